"""GPU parity: tensor-core operand forms (prepack), the product on prepared operands, chained form outputs."""
import numpy as np
import pytest
import torch

import oracle
from util import Guarded, as_i32_words, dev, pack_bits_ref, unpack_words, words_np, words_per_row

pytestmark = pytest.mark.gpu

E2M1 = {0: 0x0, 1: 0x2, 2: 0x4, 3: 0x5, -1: 0xA, -2: 0xC, -3: 0xD}


@pytest.fixture(scope="module")
def q():
    import paper_1609_07061_b200.binding as b
    return b


def _planes_ref(codes, bits, ld):
    return np.stack([pack_bits_ref(((codes >> i) & 1).astype(np.uint8), ld) for i in range(bits)])


def _values(codes, bits, mode):
    return codes.astype(np.int32) if mode == 0 else (2 * codes.astype(np.int32) - ((1 << bits) - 1))


def form_ref(values, K, form, q):
    """Test-side encoding of integer values [rows, K] in a tensor-core form (independent of the library)."""
    rows = values.shape[0]
    kp = words_per_row(K) * 32
    v = np.zeros((rows, kp), np.int32)
    v[:, :K] = values
    if form == q.QNN_FORM_I8:
        return (v & 0xff).astype(np.uint8)
    nib = np.vectorize(E2M1.__getitem__)(v).astype(np.uint8)
    return (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8)


@pytest.mark.parametrize("planes,mode,form_name", [(1, 1, "FP4"), (1, 0, "FP4"), (2, 0, "FP4"), (2, 1, "FP4"),
                                                   (1, 1, "I8"), (8, 0, "I8"), (4, 1, "I8"), (7, 1, "I8"), (3, 0, "I8")])
@pytest.mark.parametrize("rows,K", [(1, 1), (5, 31), (7, 33), (130, 784), (33, 1000)])
def test_prepack_matches_reference_encoding(q, planes, mode, form_name, rows, K):
    form = getattr(q, "QNN_FORM_" + form_name)
    rng = np.random.default_rng(rows * 31 + K + planes * 7 + mode)
    codes = rng.integers(0, 1 << planes, (rows, K)).astype(np.int32)
    ld = words_per_row(K) + 2
    pl = _planes_ref(codes, planes, ld)
    rb = words_per_row(K) * (32 if form == q.QNN_FORM_I8 else 16)      # bytes the elements need
    assert q.qnn_tc_row_bytes(K, form) == (rb + 127) // 128 * 128     # recommended pitch: whole 128-byte lines
    ldb = rb + 16
    out = Guarded((rows, ldb), torch.uint8, fill=0x5C)
    q.qnn_tc_prepack(as_i32_words(pl).cuda(), planes, mode, ld, rows * ld, rows, K, form, out.t, ldb)
    torch.cuda.synchronize()
    got = out.t.cpu().numpy()
    np.testing.assert_array_equal(got[:, :rb], form_ref(_values(codes, planes, mode), K, form, q))
    assert (got[:, rb:] == 0x5C).all()
    out.check()


def test_prepack_rejects_values_that_do_not_fit(q):
    out = torch.zeros(64, dtype=torch.uint8, device="cuda")
    pl = torch.zeros(8, 1, 1, dtype=torch.int32, device="cuda")
    for planes, mode, form in [(3, 0, q.QNN_FORM_FP4), (3, 1, q.QNN_FORM_FP4), (8, 1, q.QNN_FORM_I8)]:
        with pytest.raises(q.QnnError) as ei:
            q.qnn_tc_prepack(pl, planes, mode, 1, 1, 1, 32, form, out, 32)
        assert ei.value.status == q.QNN_ERR_UNSUPPORTED
    assert q.qnn_tc_form(1, 1, 1, 1, 4096) == q.QNN_FORM_FP4
    assert q.qnn_tc_form(2, 0, 1, 1, 9216) == q.QNN_FORM_FP4
    assert q.qnn_tc_form(1, 1, 1, 1, 1 << 24) == q.QNN_FORM_I8       # fp32 sums would no longer be exact
    assert q.qnn_tc_form(4, 1, 4, 1, 2048) == q.QNN_FORM_I8
    assert q.qnn_tc_form(8, 1, 1, 1, 64) == 0


@pytest.mark.parametrize("form_name", ["FP4", "I8"])
@pytest.mark.parametrize("out_form_name", ["FP4", "I8"])
@pytest.mark.parametrize("M,N,K", [(5, 7, 33), (130, 257, 800), (300, 96, 4096), (129, 1000, 96)])
def test_tc_gemm_all_outputs(q, form_name, out_form_name, M, N, K):
    """int32, packed bits and form output of one call, prepared operands, ragged shapes."""
    form = getattr(q, "QNN_FORM_" + form_name)
    oform = getattr(q, "QNN_FORM_" + out_form_name)
    rng = np.random.default_rng(M + 3 * N + 5 * K)
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    s = oracle.xnor_gemm(X, W)
    T = rng.integers(-20, 21, N).astype(np.int32)
    T[::4] = s[0, ::4]
    flip = rng.integers(0, 2, N).astype(np.uint8)
    ld = words_per_row(K)
    a = as_i32_words(pack_bits_ref((X >= 0).astype(np.uint8), ld)).cuda()
    b = as_i32_words(pack_bits_ref((W >= 0).astype(np.uint8).T, ld)).cuda()
    rb = q.qnn_tc_row_bytes(K, form)
    af = torch.empty(M, rb, dtype=torch.uint8, device="cuda")
    bf = torch.empty(N, rb + 32, dtype=torch.uint8, device="cuda")
    q.qnn_tc_prepack(a, 1, 1, ld, 0, M, K, form, af, rb)
    q.qnn_tc_prepack(b, 1, 1, ld, 0, N, K, form, bf, rb + 32)
    out = Guarded((M, N + 1), torch.int32, fill=-7)
    ldw = words_per_row(N) + 1
    bits = Guarded((M, ldw), torch.int32, fill=0x77777777)
    orb = q.qnn_tc_row_bytes(N, oform)
    onb = words_per_row(N) * (32 if oform == q.QNN_FORM_I8 else 16)       # bytes the N outputs occupy
    of = Guarded((M, orb + 16), torch.uint8, fill=0x5C)
    q.qnn_tc_gemm(q.tc_operand(af, rb, form), q.tc_operand(bf, rb + 32, form), M, N, K, out.t, N + 1, dev(T), dev(flip),
                  bits.t, ldw, of.t, oform, orb + 16)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    np.testing.assert_array_equal(out.t.cpu().numpy()[:, :N], s)
    assert (out.t.cpu().numpy()[:, N:] == -7).all()
    want_bits = oracle.threshold(s, T, flip)
    np.testing.assert_array_equal(unpack_words(words_np(bits.t), N), want_bits)
    assert (words_np(bits.t)[:, words_per_row(N):] == 0x77777777).all()
    got_f = of.t.cpu().numpy()
    np.testing.assert_array_equal(got_f[:, :onb], form_ref(2 * want_bits.astype(np.int32) - 1, N, oform, q))
    assert (got_f[:, onb:] == 0x5C).all()
    for g in (out, bits, of):
        g.check()


@pytest.mark.parametrize("form_name", ["FP4", "I8"])
def test_tc_gemm_chain_two_layers(q, form_name):
    """Hidden layer -> form output -> next product, without ever materialising packed bits."""
    form = getattr(q, "QNN_FORM_" + form_name)
    rng = np.random.default_rng(17)
    M, K, H, N = 200, 300, 500, 70
    X = rng.standard_normal((M, K)).astype(np.float32)
    W1 = rng.uniform(-1, 1, (K, H)).astype(np.float32)
    W2 = rng.uniform(-1, 1, (H, N)).astype(np.float32)
    T = rng.integers(-10, 11, H).astype(np.int32)
    s1 = oracle.xnor_gemm(X, W1)
    h = 2.0 * oracle.threshold(s1, T, None).astype(np.float32) - 1.0
    want = oracle.xnor_gemm(h, W2)

    def prep(bits01, rows, KK):
        ld = words_per_row(KK)
        w = as_i32_words(pack_bits_ref(bits01, ld)).cuda()
        rb = q.qnn_tc_row_bytes(KK, form)
        o = torch.empty(rows, rb, dtype=torch.uint8, device="cuda")
        q.qnn_tc_prepack(w, 1, 1, ld, 0, rows, KK, form, o, rb)
        return o, rb

    af, rba = prep((X >= 0).astype(np.uint8), M, K)
    w1f, _ = prep((W1 >= 0).astype(np.uint8).T, H, K)
    w2f, rbh = prep((W2 >= 0).astype(np.uint8).T, N, H)
    hf = torch.empty(M, rbh, dtype=torch.uint8, device="cuda")
    q.qnn_tc_gemm(q.tc_operand(af, rba, form), q.tc_operand(w1f, rba, form), M, H, K, thr=dev(T), out_form=hf,
                  out_form_kind=form, ld_form_bytes=rbh)
    out = torch.empty(M, N, dtype=torch.int32, device="cuda")
    q.qnn_tc_gemm(q.tc_operand(hf, rbh, form), q.tc_operand(w2f, rbh, form), M, N, H, out, N)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0
    np.testing.assert_array_equal(out.cpu().numpy(), want)


@pytest.mark.parametrize("K", [65536, 1 << 20])
def test_fp4_accumulation_exact_at_large_sums(q, K):
    """Closed forms at sums far beyond fp16/bf16 range: all-agree rows give +K, all-disagree -K, half-and-half 0."""
    form = q.QNN_FORM_FP4
    M, N = 4, 40
    ld = K // 32
    a = np.zeros((M, ld), np.uint32)
    a[0, :] = 0xffffffff                                  # all +1
    a[1, :] = 0                                           # all -1
    a[2, : ld // 2] = 0xffffffff                          # first half +1
    a[3, :] = 0x55555555
    b = np.full((N, ld), 0xffffffff, np.uint32)           # all +1
    b[1, :] = 0
    b[2, :] = 0xaaaaaaaa
    rb = q.qnn_tc_row_bytes(K, form)
    af = torch.empty(M, rb, dtype=torch.uint8, device="cuda")
    bf = torch.empty(N, rb, dtype=torch.uint8, device="cuda")
    q.qnn_tc_prepack(as_i32_words(a).cuda(), 1, 1, ld, 0, M, K, form, af, rb)
    q.qnn_tc_prepack(as_i32_words(b).cuda(), 1, 1, ld, 0, N, K, form, bf, rb)
    out = torch.empty(M, N, dtype=torch.int32, device="cuda")
    q.qnn_tc_gemm(q.tc_operand(af, rb, form), q.tc_operand(bf, rb, form), M, N, K, out, N)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert got[0, 0] == K and got[1, 0] == -K and got[2, 0] == 0 and got[3, 0] == 0
    assert got[0, 1] == -K and got[1, 1] == K
    assert got[3, 2] == -K and got[0, 2] == 0
    assert (got[0, 3:] == K).all()


def test_tc_gemm_argument_errors(q):
    t = torch.zeros(256, dtype=torch.uint8, device="cuda")
    o = torch.zeros(16, dtype=torch.int32, device="cuda")
    a = q.tc_operand(t, 16, q.QNN_FORM_FP4)
    b8 = q.tc_operand(t, 32, q.QNN_FORM_I8)
    with pytest.raises(q.QnnError) as ei:
        q.qnn_tc_gemm(a, b8, 2, 2, 32, o, 2)
    assert ei.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as ei:
        q.qnn_tc_gemm(a, a, 2, 2, 32)                      # no output
    assert ei.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as ei:
        q.qnn_tc_gemm(a, a, 2, 2, 64, o, 2)                # rows of 16 bytes cannot hold K = 64
    assert ei.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as ei:
        q.qnn_tc_gemm(q.tc_operand(t, 16, q.QNN_FORM_FP4, planes=3), a, 2, 2, 32, o, 2)
    assert ei.value.status == q.QNN_ERR_UNSUPPORTED


@pytest.mark.parametrize("form_name,M,N,K", [("FP4", 4100, 1000, 4100), ("FP4", 5000, 777, 3104), ("I8", 4400, 900, 1600),
                                                 ("FP4", 4100, 901, 3200), ("I8", 4400, 1029, 1600), ("FP4", 4100, 1137, 3104),
                                                 ("I8", 8300, 1100, 800), ("I8", 8300, 1030, 520)])
@pytest.mark.parametrize("outputs", ["int", "sign"])
def test_tc_gemm_cta_pair_shapes(q, form_name, M, N, K, outputs):
    """Ragged shapes large enough (and with K long enough) for the product to run on CTA pairs: 256-row tiles whose
    second half hangs over the end of M, a last column tile of a few columns (5, 17, 104 ...: the kernel narrows the
    last block's instructions to the next multiple of 16), a partial last K block; the int8 shapes with K = 800 and 520 run
    on the short-K pairs (three epilogue warps per accumulator quarter).  The oracle
    runs on sampled rows (every row position inside a pair's tile is hit) and row-sum checksums cover all outputs."""
    form = getattr(q, "QNN_FORM_" + form_name)
    rng = np.random.default_rng(M + N + K)
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    ld = words_per_row(K)
    a = as_i32_words(pack_bits_ref((X >= 0).astype(np.uint8), ld)).cuda()
    b = as_i32_words(pack_bits_ref((W >= 0).astype(np.uint8).T, ld)).cuda()
    rb = q.qnn_tc_row_bytes(K, form)
    af = torch.empty(M, rb, dtype=torch.uint8, device="cuda")
    bf = torch.empty(N, rb, dtype=torch.uint8, device="cuda")
    q.qnn_tc_prepack(a, 1, 1, ld, 0, M, K, form, af, rb)
    q.qnn_tc_prepack(b, 1, 1, ld, 0, N, K, form, bf, rb)
    rows = np.unique(np.concatenate([np.arange(0, 260), np.arange(M - 300, M), rng.integers(0, M, 64)]))
    want = oracle.xnor_gemm(X[rows], W)
    A, B = q.tc_operand(af, rb, form), q.tc_operand(bf, rb, form)
    if outputs == "int":
        out = Guarded((M, N), torch.int32, fill=-7)
        q.qnn_tc_gemm(A, B, M, N, K, out.t, N)
        torch.cuda.synchronize()
        assert q.qnn_device_status() == 0, q.qnn_last_error()
        got = out.t.cpu().numpy()
        np.testing.assert_array_equal(got[rows], want)
        sa = np.where(X >= 0, 1, -1).astype(np.int64)
        sw = np.where(W >= 0, 1, -1).astype(np.int64)
        np.testing.assert_array_equal(got.sum(axis=1, dtype=np.int64), sa @ sw.sum(axis=1))
        out.check()
    else:
        T = rng.integers(-30, 31, N).astype(np.int32)
        flip = rng.integers(0, 2, N).astype(np.uint8)
        ldw = words_per_row(N)
        bits = Guarded((M, ldw), torch.int32, fill=0)
        orb = q.qnn_tc_row_bytes(N, q.QNN_FORM_FP4)
        of = Guarded((M, orb), torch.uint8, fill=0x5C)
        q.qnn_tc_gemm(A, B, M, N, K, thr=dev(T), flip=dev(flip), out_bits=bits.t, ld_words=ldw, out_form=of.t,
                      out_form_kind=q.QNN_FORM_FP4, ld_form_bytes=orb)
        torch.cuda.synchronize()
        assert q.qnn_device_status() == 0, q.qnn_last_error()
        wb = oracle.threshold(want, T, flip)
        np.testing.assert_array_equal(unpack_words(words_np(bits.t)[rows], N), wb)
        onb = words_per_row(N) * 16
        np.testing.assert_array_equal(of.t.cpu().numpy()[rows][:, :onb], form_ref(2 * wb.astype(np.int32) - 1, N, q.QNN_FORM_FP4, q))
        bits.check(); of.check()


@pytest.mark.parametrize("M,N,K,la,lb", [(70, 40, 96, (-3, 3), None), (300, 130, 1000, (-2, 1), (-1, 2)), (129, 257, 4096, (-6, 0), (-3, 3)),
                                          (5, 3, 31, (0, 0), (0, 2))])
def test_logquant_products(q, M, N, K, la, lb):
    """Logarithmically quantised activations (Eq. 10) times +-1 or logarithmically quantised weights on the int8
    tensor-core form: exact integer sums in units of the two smallest levels."""
    rng = np.random.default_rng(M + N + K)
    X = (rng.standard_normal((M, K)) * 2.0).astype(np.float32)
    Wt = (rng.standard_normal((N, K)) * 0.7).astype(np.float32)          # weights, one row per unit
    va = oracle.log_quant(X, *la)
    kz = (K + 31) // 32 * 32
    ld = (kz + 15) // 16 * 16
    a8 = torch.zeros(M, ld, dtype=torch.uint8, device="cuda")
    q.qnn_logquant_pack_i8(dev(X), M, K, K, la[0], la[1], a8, ld)
    b8 = torch.zeros(N, ld, dtype=torch.uint8, device="cuda")
    if lb is None:
        vb = oracle.sign(Wt)
        bits = torch.zeros(N, (K + 31) // 32, dtype=torch.int32, device="cuda")
        q.qnn_quantize_pack_sign(dev(Wt), N, K, K, bits, (K + 31) // 32)
        q.qnn_tc_prepack(bits, 1, q.QNN_MODE_PM1, (K + 31) // 32, 0, N, K, q.QNN_FORM_I8, b8, ld)
        pb = 1
    else:
        vb = oracle.log_quant(Wt, *lb)
        q.qnn_logquant_pack_i8(dev(Wt), N, K, K, lb[0], lb[1], b8, ld)
        pb = lb[1] - lb[0] + 1
    want = oracle.int_gemm(va, vb.T)
    out = Guarded((M, N), torch.int32, fill=-7)
    A = q.tc_operand(a8, ld, q.QNN_FORM_I8, planes=la[1] - la[0] + 1, mode=q.QNN_MODE_PM1)
    Bo = q.tc_operand(b8, ld, q.QNN_FORM_I8, planes=pb, mode=q.QNN_MODE_PM1)
    q.qnn_tc_gemm(A, Bo, M, N, K, out=out.t, ldo=N)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    np.testing.assert_array_equal(out.t.cpu().numpy(), want)
    out.check()


def _log_backward_product(q, G_f32, transposed, rows, K, W_pm1_rows, emin, emax):
    """LogQuant(gradient) [rows, K] times +-1 rows [N, K] -> int64 [rows, N] through the group operand, one int8 product and
    the combine step.  G_f32: the gradient as stored ([rows, K], or [K, rows] when `transposed`)."""
    N = W_pm1_rows.shape[0]
    groups = q.qnn_logquant_groups(emin, emax)
    kz = (K + 31) // 32 * 32
    ld = (kz + 15) // 16 * 16
    a8 = Guarded((groups * rows, ld), torch.uint8, fill=0x5C)
    q.qnn_logquant_pack_groups(dev(G_f32), rows, K, G_f32.shape[1], transposed, emin, emax, a8.t, ld)
    bits = torch.zeros(N, (K + 31) // 32, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_sign(dev(W_pm1_rows.astype(np.float32)), N, K, K, bits, (K + 31) // 32)
    b8 = torch.zeros(N, ld, dtype=torch.uint8, device="cuda")
    q.qnn_tc_prepack(bits, 1, q.QNN_MODE_PM1, (K + 31) // 32, 0, N, K, q.QNN_FORM_I8, b8, ld)
    part = torch.empty(groups * rows, N, dtype=torch.int32, device="cuda")
    A = q.tc_operand(a8.t, ld, q.QNN_FORM_I8, planes=7, mode=q.QNN_MODE_PM1)
    Bo = q.tc_operand(b8, ld, q.QNN_FORM_I8, planes=1, mode=q.QNN_MODE_PM1)
    q.qnn_tc_gemm(A, Bo, groups * rows, N, K, out=part, ldo=N)
    out = Guarded((rows, N), torch.int64, fill=-7)
    q.qnn_logquant_combine(part, groups, rows, N, N, out.t, N)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    a8.check(); out.check()
    return a8.t.cpu().numpy().view(np.int8), out.t.cpu().numpy()


@pytest.mark.parametrize("M,Nu,K,emin,emax", [(70, 40, 96, -30, 0), (300, 130, 1000, -20, -3), (129, 257, 515, -6, 0), (33, 5, 31, -14, 0)])
def test_alg1_backward_products_log_gradients(q, M, Nu, K, emin, emax):
    """Algorithm 1's backward pass with logarithmically quantised gradients (Eq. 10, up to 31 exponents: the 6-bit code of
    Sec. 4.4): g_a = LogQuant(g_s) W^b (batch x units times units x inputs) and g_W = a^b^T LogQuant(g_s), the second one
    contracting over the batch through the transposed packer.  Exact int64 sums against the oracle; the group operand's
    bytes against the oracle's codes."""
    rng = np.random.default_rng(M + Nu + K)
    gs = (rng.standard_normal((M, Nu)) * np.exp2(rng.integers(emin - 2, emax + 3, (M, Nu)))).astype(np.float32)   # gradient of the layer's sums
    gs.reshape(-1)[:7] = np.array([0.0, -0.0, np.nan, np.inf, -np.inf, 1e-45, -1e-45], np.float32)
    Wb = rng.integers(0, 2, (K, Nu)).astype(np.int32) * 2 - 1          # the layer's +-1 weights [inputs, units]
    ab = rng.integers(0, 2, (M, K)).astype(np.int32) * 2 - 1           # its +-1 input activations
    # g_a[m, k] = sum_n LogQuant(g_s)[m, n] W[k, n]: contraction over the units; the gradient's rows are operand rows
    codes, got_a = _log_backward_product(q, gs, 0, M, Nu, Wb, emin, emax)
    np.testing.assert_array_equal(got_a, oracle.log_gemm(gs, Wb.T, emin, emax))
    v = oracle.log_quant(gs, emin, emax).astype(np.int64)
    groups = q.qnn_logquant_groups(emin, emax)
    rebuilt = sum(codes[g * M:(g + 1) * M, :Nu].astype(np.int64) << (7 * g) for g in range(groups))
    np.testing.assert_array_equal(rebuilt, v)
    assert (codes[:, Nu:(Nu + 31) // 32 * 32] == 0).all()
    # g_W[n, k] = sum_m LogQuant(g_s)[m, n] a[m, k]: contraction over the batch; the gradient's COLUMNS are operand rows
    _, got_w = _log_backward_product(q, gs, 1, Nu, M, np.ascontiguousarray(ab.T), emin, emax)
    np.testing.assert_array_equal(got_w, oracle.log_gemm(np.ascontiguousarray(gs.T), ab, emin, emax))


def test_logquant_groups_argument_errors(q):
    x = torch.zeros(4, 32, device="cuda")
    out = torch.zeros(5 * 4, 32, dtype=torch.uint8, device="cuda")
    assert q.qnn_logquant_groups(-30, 0) == 5 and q.qnn_logquant_groups(-6, 0) == 1 and q.qnn_logquant_groups(-7, 0) == 2
    assert q.qnn_logquant_groups(-31, 0) == 0 and q.qnn_logquant_groups(1, 0) == 0
    with pytest.raises(q.QnnError) as e:
        q.qnn_logquant_pack_groups(x, 4, 32, 32, 0, -31, 0, out, 32)
    assert e.value.status == q.QNN_ERR_UNSUPPORTED
    with pytest.raises(q.QnnError) as e:
        q.qnn_logquant_pack_groups(x, 4, 32, 16, 0, -3, 0, out, 32)          # ldx below K
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as e:
        q.qnn_logquant_pack_groups(x, 4, 32, 32, 0, -3, 0, out, 30)          # row stride below K rounded up
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    p = torch.zeros(8, 4, dtype=torch.int32, device="cuda")
    o = torch.zeros(4, 4, dtype=torch.int64, device="cuda")
    with pytest.raises(q.QnnError) as e:
        q.qnn_logquant_combine(p, 6, 4, 4, 4, o, 4)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    q.qnn_logquant_pack_groups(x, 0, 32, 32, 0, -3, 0, out, 32)              # empty: nothing to do
    q.qnn_logquant_combine(p, 2, 0, 4, 4, o, 4)


@pytest.mark.parametrize("K", [256, 512, 200])
@pytest.mark.parametrize("a_rows", ["zeros", "mixed"])
def test_fp4_zero_sum_against_zero_threshold(q, K, a_rows):
    """An all-zero 2-bit activation row against all -1 weights sums products 0 * (-1): in fp32 the accumulator may
    come out as -0.0.  Eq. 1 gives sign(0) = +1, so with threshold 0 the bit must be 1 whatever the zero's sign
    (bits and form output; the oracle decides on integers)."""
    M, N = 130, 70
    rng = np.random.default_rng(K)
    codes = np.zeros((M, K), np.int32) if a_rows == "zeros" else rng.integers(0, 4, (M, K)).astype(np.int32)
    codes[::3] = 0                                               # whole rows of zeros among the others
    wsign = -np.ones((K, N), np.int32)
    if a_rows == "mixed":
        wsign[:, 1::2] = np.where(rng.random((K, (N + 0) // 2)) < 0.5, 1, -1)
    s = oracle.int_gemm(codes, wsign)
    T = np.zeros(N, np.int32)
    flip = np.zeros(N, np.uint8); flip[5::7] = 1
    ld = words_per_row(K)
    pl = _planes_ref(codes, 2, ld)
    a = as_i32_words(pl).cuda()
    b = as_i32_words(pack_bits_ref((wsign.T > 0).astype(np.uint8), ld)).cuda()
    form = q.QNN_FORM_FP4
    rb = q.qnn_tc_row_bytes(K, form)
    af = torch.empty(M, rb, dtype=torch.uint8, device="cuda")
    bf = torch.empty(N, rb, dtype=torch.uint8, device="cuda")
    q.qnn_tc_prepack(a, 2, q.QNN_MODE_U01, ld, M * ld, M, K, form, af, rb)
    q.qnn_tc_prepack(b, 1, q.QNN_MODE_PM1, ld, 0, N, K, form, bf, rb)
    ldw = words_per_row(N)
    bits = Guarded((M, ldw), torch.int32, fill=0)
    orb = q.qnn_tc_row_bytes(N, form)
    of = Guarded((M, orb), torch.uint8, fill=0x5C)
    out = Guarded((M, N), torch.int32, fill=-7)
    q.qnn_tc_gemm(q.tc_operand(af, rb, form, 2, q.QNN_MODE_U01), q.tc_operand(bf, rb, form), M, N, K, out.t, N, dev(T), dev(flip),
                  bits.t, ldw, of.t, form, orb)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    np.testing.assert_array_equal(out.t.cpu().numpy(), s)
    want_bits = oracle.threshold(s, T, flip)
    assert want_bits[0, 0] == 1                                  # 0 >= 0
    np.testing.assert_array_equal(unpack_words(words_np(bits.t), N), want_bits)
    onb = words_per_row(N) * 16
    np.testing.assert_array_equal(of.t.cpu().numpy()[:, :onb], form_ref(2 * want_bits.astype(np.int32) - 1, N, form, q))
    for g in (out, bits, of):
        g.check()


def test_bounded_wait_that_runs_out_is_reported_once_and_leaves_the_context_usable(q):
    """Failure path of the device-side waits, provoked in the one harmless way: a diagnostic kernel polls a barrier
    that nothing arrives on (no copy, no tensor-core work in flight) until its short limit runs out.  The status word
    must report QNN_ERR_TIMEOUT exactly once, and a product right after must be bit-exact."""
    assert q.qnn_device_status() == 0
    q.qnn_selftest_wait_timeout()
    assert q.qnn_device_status() == q.QNN_ERR_TIMEOUT
    assert "wait" in q.qnn_last_error()
    assert q.qnn_device_status() == 0
    M, N, K = 200, 300, 1000
    rng = np.random.default_rng(3)
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    ld = words_per_row(K)
    a = as_i32_words(pack_bits_ref((X >= 0).astype(np.uint8), ld)).cuda()
    b = as_i32_words(pack_bits_ref((W >= 0).astype(np.uint8).T, ld)).cuda()
    out = torch.empty(M, N, dtype=torch.int32, device="cuda")
    ws = torch.empty(q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, q.QNN_ALGO_TC_FP4), dtype=torch.uint8, device="cuda")
    q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, out, N, q.QNN_ALGO_TC_FP4, ws)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0
    np.testing.assert_array_equal(out.cpu().numpy(), oracle.xnor_gemm(X, W))


def test_auto_leaves_a_note_when_it_cannot_use_the_workspace(q):
    """QNN_ALGO_AUTO with no (or a misaligned) workspace still gives the right integers on another kernel, and says so."""
    M, N, K = 300, 4096, 4096
    assert q.qnn_select_algo(M, N, K) in (q.QNN_ALGO_TC_FP4, q.QNN_ALGO_TC_I8)
    g = torch.Generator(device="cuda").manual_seed(1)
    ld = K // 32
    a = torch.randint(-2**31, 2**31 - 1, (M, ld), dtype=torch.int32, device="cuda", generator=g)
    b = torch.randint(-2**31, 2**31 - 1, (N, ld), dtype=torch.int32, device="cuda", generator=g)
    want = torch.empty(M, N, dtype=torch.int32, device="cuda")
    q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, want, N, q.QNN_ALGO_POPC)
    need = q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, q.QNN_ALGO_AUTO)
    raw = torch.empty(need + 512, dtype=torch.uint8, device="cuda")
    off = (-raw.data_ptr()) % 256
    for ws in (None, raw[off + 16: off + 16 + need]):
        got = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
        q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, got, N, q.QNN_ALGO_AUTO, ws)
        assert "instead of the tensor-core kernel on rewritten operands" in q.qnn_last_error()
        torch.cuda.synchronize()
        assert torch.equal(got, want)
