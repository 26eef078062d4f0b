"""GPU parity: quantise + pack kernels against the oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_1609_07061_b200 import workloads
from util import Guarded, dev, unpack_words, words_np, words_per_row

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q():
    import paper_1609_07061_b200.binding as b
    return b


def _special_values(n, rng):
    x = rng.standard_normal(n).astype(np.float32)
    sp = np.array([0.0, -0.0, np.nan, np.inf, -np.inf, 1e-45, -1e-45, 1.17549435e-38, -1.17549435e-38], np.float32)
    idx = rng.choice(n, size=min(n, 64), replace=False)
    x[idx] = sp[np.arange(len(idx)) % len(sp)]
    return x


@pytest.mark.parametrize("rows,K,ldx,ldw", [(1, 1, 1, 1), (3, 31, 31, 1), (5, 32, 32, 1), (7, 33, 36, 2), (4, 127, 127, 5),
                                            (9, 129, 132, 8), (2, 511, 512, 16), (13, 513, 513, 17), (64, 4096, 4096, 128),
                                            (3, 5000, 5000, 160), (100, 784, 784, 28)])
def test_pack_sign_rowmajor(q, rows, K, ldx, ldw):
    rng = np.random.default_rng(rows * 7919 + K)
    x = _special_values(rows * ldx, rng).reshape(rows, ldx)
    out = Guarded((rows, ldw), torch.int32, fill=0x5a5a5a5a)
    popc = Guarded((rows,), torch.int32, fill=-1)
    q.qnn_quantize_pack_sign(dev(x), rows, K, ldx, out.t, ldw, popc.t)
    torch.cuda.synchronize()
    want = (oracle.sign(x[:, :K]) > 0).astype(np.uint8)
    got = unpack_words(words_np(out.t), K)
    np.testing.assert_array_equal(got, want)
    np.testing.assert_array_equal(popc.t.cpu().numpy(), want.sum(axis=1))
    # words beyond ceil(K/32) are untouched
    assert (words_np(out.t)[:, words_per_row(K):] == 0x5a5a5a5a).all()
    out.check(); popc.check()


def test_pack_sign_unaligned_base(q):
    """A source pointer that is only 4-byte aligned takes the scalar path and gives the same bits."""
    rng = np.random.default_rng(5)
    rows, K = 6, 200
    buf = dev(_special_values(rows * K + 1, rng))
    x = buf[1:]
    out = torch.zeros(rows, 7, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_sign(x, rows, K, K, out, 7)
    want = (oracle.sign(x.cpu().numpy().reshape(rows, K)) > 0).astype(np.uint8)
    np.testing.assert_array_equal(unpack_words(words_np(out), K), want)


@pytest.mark.parametrize("K,N,ldw_in,ld", [(1, 1, 1, 1), (31, 5, 5, 1), (33, 7, 8, 2), (64, 130, 130, 2), (100, 129, 132, 4),
                                           (784, 4096, 4096, 28), (4096, 10, 10, 128), (300, 1000, 1000, 12)])
def test_pack_sign_transposed(q, K, N, ldw_in, ld):
    rng = np.random.default_rng(K * 31 + N)
    w = _special_values(K * ldw_in, rng).reshape(K, ldw_in)
    out = Guarded((N, ld), torch.int32, fill=0)
    popc = Guarded((N,), torch.int32, fill=-1)
    q.qnn_quantize_pack_sign_t(dev(w), K, N, ldw_in, out.t, ld, popc.t)
    torch.cuda.synchronize()
    want = (oracle.sign(w[:, :N]) > 0).astype(np.uint8).T
    np.testing.assert_array_equal(unpack_words(words_np(out.t), K), want)
    np.testing.assert_array_equal(popc.t.cpu().numpy(), want.sum(axis=1))
    out.check(); popc.check()


@pytest.mark.parametrize("B,C,H,W", [(1, 1, 1, 1), (2, 3, 5, 7), (2, 33, 4, 4), (3, 256, 16, 16), (1, 70, 3, 9)])
def test_pack_sign_nchw(q, B, C, H, W):
    rng = np.random.default_rng(B + C + H + W)
    x = _special_values(B * C * H * W, rng).reshape(B, C, H, W)
    cw = words_per_row(C)
    out = Guarded((B, H, W, cw), torch.int32, fill=0)
    q.qnn_quantize_pack_sign_nchw(dev(x), B, C, H, W, out.t)
    torch.cuda.synchronize()
    want = (oracle.sign(x) > 0).astype(np.uint8).transpose(0, 2, 3, 1).reshape(-1, C)
    np.testing.assert_array_equal(unpack_words(words_np(out.t).reshape(-1, cw), C), want)
    out.check()


@pytest.mark.parametrize("bits,lo,hi", [(1, -1.0, 1.0), (2, 0.0, 1.0), (4, -1.0, 1.0), (8, 0.0, 1.0), (3, -3.0, 5.0)])
@pytest.mark.parametrize("rows,K", [(1, 1), (5, 33), (9, 128), (4, 130), (256, 1000)])
def test_quantize_kbit_rowmajor(q, bits, lo, hi, rows, K):
    rng = np.random.default_rng(bits * 100 + rows + K)
    x = (rng.standard_normal((rows, K)) * 0.7).astype(np.float32)
    L = (1 << bits) - 1
    # exact level centres, exact ties of the fp32 quotient where representable, and specials
    x.flat[: min(x.size, L + 1)] = (lo + np.arange(min(x.size, L + 1)) * (hi - lo) / L).astype(np.float32)
    if x.size > 40:
        x.flat[20:26] = [np.nan, np.inf, -np.inf, lo, hi, -0.0]
    ld = words_per_row(K) + 1
    stride = rows * ld + 3
    planes = Guarded((bits * stride,), torch.int32, fill=0)
    rs = Guarded((rows,), torch.int32, fill=-1)
    q.qnn_quantize_pack_kbit(dev(x), rows, K, K, bits, lo, hi, planes.t, ld, stride, rs.t)
    torch.cuda.synchronize()
    want = oracle.linear_quant_codes(x, bits, lo, hi)
    pw = words_np(planes.t)
    got = np.zeros((rows, K), np.int32)
    for i in range(bits):
        plane = pw[i * stride: i * stride + rows * ld].reshape(rows, ld)
        bits_i = unpack_words(plane, K)
        np.testing.assert_array_equal(bits_i, oracle.bit_plane(want, i))
        got += bits_i.astype(np.int32) << i
    np.testing.assert_array_equal(got, want)
    np.testing.assert_array_equal(rs.t.cpu().numpy(), want.sum(axis=1))
    planes.check(); rs.check()


def test_quantize_kbit_ties(q):
    # lo = 0, hi = 15, 4 bits: the step is exactly 1, so j + 0.5 ties are exact in fp32
    x = (np.arange(0, 15, dtype=np.float32) + 0.5).reshape(1, 15)
    planes = torch.zeros(4, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_kbit(dev(x), 1, 15, 15, 4, 0.0, 15.0, planes, 1, 1)
    pw = words_np(planes)
    got = sum((unpack_words(pw[i:i + 1].reshape(1, 1), 15).astype(np.int32) << i) for i in range(4))
    np.testing.assert_array_equal(got, oracle.linear_quant_codes(x, 4, 0.0, 15.0))
    np.testing.assert_array_equal(got[0], [0, 2, 2, 4, 4, 6, 6, 8, 8, 10, 10, 12, 12, 14, 14])


@pytest.mark.parametrize("bits", [1, 2, 4, 8])
@pytest.mark.parametrize("K,N", [(1, 1), (33, 5), (100, 130), (2048, 512)])
def test_quantize_kbit_transposed(q, bits, K, N):
    rng = np.random.default_rng(bits + K + N)
    w = rng.uniform(-1.2, 1.2, (K, N)).astype(np.float32)
    ld = words_per_row(K)
    stride = N * ld
    planes = Guarded((bits, N, ld), torch.int32, fill=0)
    rs = Guarded((N,), torch.int32, fill=-1)
    q.qnn_quantize_pack_kbit_t(dev(w), K, N, N, bits, -1.0, 1.0, planes.t, ld, stride, rs.t)
    torch.cuda.synchronize()
    want = oracle.linear_quant_codes(w, bits, -1.0, 1.0).T
    pw = words_np(planes.t)
    for i in range(bits):
        np.testing.assert_array_equal(unpack_words(pw[i], K), oracle.bit_plane(want, i))
    np.testing.assert_array_equal(rs.t.cpu().numpy(), want.sum(axis=1))
    planes.check(); rs.check()


@pytest.mark.parametrize("bits", [8, 4, 1])
@pytest.mark.parametrize("rows,K,ldx", [(1, 1, 1), (7, 31, 33), (10, 784, 784), (3, 1000, 1024)])
def test_pack_planes_u8(q, bits, rows, K, ldx):
    rng = np.random.default_rng(rows + K)
    x = rng.integers(0, 256, (rows, ldx)).astype(np.uint8)
    ld = (words_per_row(K) + 3) // 4 * 4
    stride = rows * ld
    planes = Guarded((bits, rows, ld), torch.int32, fill=0)
    rs = Guarded((rows,), torch.int32, fill=-1)
    q.qnn_pack_planes_u8(dev(x), rows, K, ldx, bits, planes.t, ld, stride, rs.t)
    torch.cuda.synchronize()
    codes = x[:, :K].astype(np.int32) % (1 << bits)
    pw = words_np(planes.t)
    for i in range(bits):
        np.testing.assert_array_equal(unpack_words(pw[i], K), oracle.bit_plane(codes, i))
    np.testing.assert_array_equal(rs.t.cpu().numpy(), codes.sum(axis=1))
    planes.check(); rs.check()


@pytest.mark.parametrize("M,N,lds", [(1, 1, 1), (5, 31, 31), (9, 33, 36), (17, 128, 128), (100, 4096, 4096), (3, 1000, 1003)])
@pytest.mark.parametrize("with_flip", [False, True])
def test_threshold_pack(q, M, N, lds, with_flip):
    rng = np.random.default_rng(M + N)
    s = rng.integers(-200, 200, (M, lds)).astype(np.int32)
    T = rng.integers(-64, 65, N).astype(np.int32)
    s[:, : min(N, lds)][:, ::3] = T[::3][None, :]            # plenty of exact equalities
    flip = rng.integers(0, 2, N).astype(np.uint8) if with_flip else None
    ld = words_per_row(N) + 2
    out = Guarded((M, ld), torch.int32, fill=0x11111111)
    q.qnn_threshold_pack(dev(s), M, N, lds, dev(T), None if flip is None else dev(flip), out.t, ld)
    torch.cuda.synchronize()
    want = oracle.threshold(s[:, :N], T, flip)
    np.testing.assert_array_equal(unpack_words(words_np(out.t), N), want)
    out.check()


def test_rescale_f32(q):
    rng = np.random.default_rng(3)
    M, N = 37, 130
    p = rng.integers(-5000, 5000, (M, N)).astype(np.int32)
    r = rng.standard_normal(M).astype(np.float32)
    c = rng.standard_normal(N).astype(np.float32)
    y = Guarded((M, N), torch.float32, fill=0)
    q.qnn_rescale_f32(dev(p), M, N, N, 0.0123, dev(r), dev(c), -0.5, y.t, N)
    torch.cuda.synchronize()
    want = oracle.rescale(p, float(np.float32(0.0123)), r.astype(np.float64), c.astype(np.float64), -0.5)
    got = y.t.cpu().numpy().astype(np.float64)
    # tolerance stated by the benchmark spec: 1e-6 relative (relative to the magnitude of the terms summed)
    scale = np.abs(np.float32(0.0123) * p) + np.abs(r)[:, None] + np.abs(c)[None, :] + 0.5
    assert np.max(np.abs(got - want) / scale) <= 1e-6
    y.check()


@pytest.mark.parametrize("rows,K,ldx,emin,emax", [(7, 100, 100, -3, 3), (64, 4096, 4096, -2, 1), (3, 33, 40, 0, 0), (129, 784, 784, -6, 0),
                                                   (5, 1, 4, -1, 2)])
def test_logquant_pack_i8(q, rows, K, ldx, emin, emax):
    """Eq. 10 / AP2: int8 values sign * 2^(e - emin) against the oracle, bit-exact; pad bytes up to 32-multiples zero."""
    rng = np.random.default_rng(rows * 7 + K)
    x = (rng.standard_normal((rows, ldx)) * np.exp(rng.uniform(-4, 4, (rows, ldx)))).astype(np.float32)
    lo = np.float32(1.41421353816986083984375)
    specials = [0.0, -0.0, np.inf, -np.inf, np.nan, 1e-40, -1e-40, lo, np.nextafter(lo, np.float32(2)), -lo, 0.5 * lo, 1.0, -1.0, 1.5, 3.0]
    flat = x.reshape(-1)
    n = min(len(specials), flat.size)
    flat[:n] = np.array(specials[:n], np.float32)
    kz = (K + 31) // 32 * 32
    ld_bytes = kz + 16
    out = Guarded((rows, ld_bytes), torch.uint8, fill=0x5C)
    q.qnn_logquant_pack_i8(dev(x), rows, K, ldx, emin, emax, out.t, ld_bytes)
    torch.cuda.synchronize()
    got = out.t.cpu().numpy()
    want = oracle.log_quant(x[:, :K], emin, emax)
    np.testing.assert_array_equal(got[:, :K].view(np.int8).astype(np.int32), want)
    assert not got[:, K:kz].any(), "bytes between K and the next multiple of 32 must be zero"
    assert (got[:, kz:] == 0x5C).all(), "bytes past the written part of a row must stay untouched"
    out.check()


def test_logquant_argument_errors(q):
    x = torch.zeros(4, 32, device="cuda")
    out = torch.zeros(4, 32, dtype=torch.uint8, device="cuda")
    with pytest.raises(q.QnnError) as e:
        q.qnn_logquant_pack_i8(x, 4, 32, 32, -4, 3, out, 32)          # 8 levels: 2^7 does not fit int8
    assert e.value.status == q.QNN_ERR_UNSUPPORTED
    with pytest.raises(q.QnnError) as e:
        q.qnn_logquant_pack_i8(x, 4, 32, 32, 2, 1, out, 32)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as e:
        q.qnn_logquant_pack_i8(x, 4, 20, 32, 0, 1, out, 20)           # row stride below K rounded up to 32
    assert e.value.status == q.QNN_ERR_INVALID_ARG


# ---- quantisers that write a tensor-core form directly ---------------------------------------------------------

_E2M1 = {0: 0x0, 1: 0x2, 2: 0x4, 3: 0x5, -1: 0xA, -2: 0xC, -3: 0xD}


def _form_bytes_of(values, K, form, q):
    """Test-side encoding of integer values [rows, K] in a tensor-core form; elements K .. next multiple of 32 are 0."""
    rows = values.shape[0]
    kp = words_per_row(K) * 32
    v = np.zeros((rows, kp), np.int32)
    v[:, :K] = values
    if form == q.QNN_FORM_I8:
        return (v & 0xff).astype(np.uint8)
    nib = np.vectorize(_E2M1.__getitem__)(v).astype(np.uint8)
    return (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8)


_SPECIALS = np.array([0.0, -0.0, 1e-45, -1e-45, np.inf, -np.inf, np.nan, 1.0, -1.0, 0.5, 1.0 / 6.0, 0.49999997, 2.5 / 3.0],
                     np.float32)


@pytest.mark.parametrize("form_name", ["FP4", "I8"])
@pytest.mark.parametrize("rows,K,ldx", [(1, 1, 1), (3, 31, 33), (5, 33, 36), (7, 1024, 1024), (130, 1000, 1000), (33, 4097, 4100), (100, 4096, 4096)])
def test_quantize_form_sign_row_major(q, rows, K, ldx, form_name):
    """Eq. 1 straight into a tensor-core form, row-major source: values +-1, pads 0, bytes past the row untouched."""
    form = getattr(q, "QNN_FORM_" + form_name)
    rng = np.random.default_rng(rows * 7 + K)
    X = rng.standard_normal((rows, ldx)).astype(np.float32)
    X.reshape(-1)[: min(X.size, _SPECIALS.size)] = _SPECIALS[: min(X.size, _SPECIALS.size)]
    eb = words_per_row(K) * (32 if form == q.QNN_FORM_I8 else 16)
    ldb = eb + 16
    out = Guarded((rows, ldb), torch.uint8, fill=0x5C)
    q.qnn_quantize_form_sign(dev(X), rows, K, ldx, form, out.t, ldb)
    torch.cuda.synchronize()
    got = out.t.cpu().numpy()
    np.testing.assert_array_equal(got[:, :eb], _form_bytes_of(oracle.sign(X[:, :K]), K, form, q))
    assert (got[:, eb:] == 0x5C).all()
    out.check()


@pytest.mark.parametrize("form_name", ["FP4", "I8"])
@pytest.mark.parametrize("K,N,ldw", [(1, 1, 1), (31, 5, 5), (33, 7, 8), (64, 130, 132), (1000, 257, 260), (4096, 512, 512), (96, 1000, 1003)])
def test_quantize_form_sign_transposed(q, K, N, ldw, form_name):
    """Weights [K, N] -> form rows [N, K] (one row per output unit), as qnn_tc_gemm's B operand wants them."""
    form = getattr(q, "QNN_FORM_" + form_name)
    rng = np.random.default_rng(K * 3 + N)
    W = rng.uniform(-1, 1, (K, ldw)).astype(np.float32)
    W.reshape(-1)[: min(W.size, _SPECIALS.size)] = _SPECIALS[: min(W.size, _SPECIALS.size)]
    eb = words_per_row(K) * (32 if form == q.QNN_FORM_I8 else 16)
    ldb = (eb + 127) // 128 * 128
    out = Guarded((N, ldb), torch.uint8, fill=0x5C)
    q.qnn_quantize_form_sign_t(dev(W), K, N, ldw, form, out.t, ldb)
    torch.cuda.synchronize()
    got = out.t.cpu().numpy()
    np.testing.assert_array_equal(got[:, :eb], _form_bytes_of(oracle.sign(W[:, :N]).T, K, form, q))
    assert (got[:, eb:] == 0x5C).all()
    out.check()


@pytest.mark.parametrize("B,C,H,W", [(2, 256, 16, 16), (3, 128, 5, 7), (1, 40, 3, 3), (2, 512, 8, 8)])
def test_quantize_form_sign_nchw(q, B, C, H, W):
    """NCHW fp32 -> NHWC pixels in e2m1 form (the implicit convolution's A operand)."""
    form = q.QNN_FORM_FP4
    rng = np.random.default_rng(B + C + H)
    X = rng.standard_normal((B, C, H, W)).astype(np.float32)
    eb = words_per_row(C) * 16
    out = Guarded((B * H * W, eb), torch.uint8, fill=0x5C)
    q.qnn_quantize_form_sign_nchw(dev(X), B, C, H, W, form, out.t, eb)
    torch.cuda.synchronize()
    want = _form_bytes_of(oracle.sign(X).transpose(0, 2, 3, 1).reshape(-1, C), C, form, q)
    np.testing.assert_array_equal(out.t.cpu().numpy(), want)
    out.check()


@pytest.mark.parametrize("bits,lo,hi,mode,form_name", [(2, 0.0, 1.0, 0, "FP4"), (2, -1.0, 1.0, 1, "FP4"), (1, -1.0, 1.0, 1, "FP4"),
                                                       (4, -1.0, 1.0, 1, "I8"), (8, 0.0, 1.0, 0, "I8"), (2, 0.0, 1.0, 0, "I8"), (3, -2.0, 5.0, 0, "I8")])
@pytest.mark.parametrize("transposed", [False, True])
def test_quantize_form_kbit(q, bits, lo, hi, mode, form_name, transposed):
    """Eq. 9 straight into a form: codes (or their signed-symmetric values) as the oracle's quantiser gives them,
    including exact ties, level centres, clipping and the special values."""
    form = getattr(q, "QNN_FORM_" + form_name)
    rows, K = (130, 1000)
    rng = np.random.default_rng(bits * 10 + mode)
    X = (rng.standard_normal((rows, K)) * (hi - lo) * 0.6 + (hi + lo) / 2).astype(np.float32)
    L = (1 << bits) - 1
    step = (hi - lo) / L
    ties = (lo + (np.arange(L) + 0.5) * step).astype(np.float32)
    X[0, :ties.size] = ties
    X[1, :L + 1] = (lo + np.arange(L + 1) * step).astype(np.float32)
    X[2, :_SPECIALS.size] = _SPECIALS
    codes = oracle.linear_quant_codes(X, bits, lo, hi)
    vals = oracle.codes_to_symmetric(codes, bits) if mode == 1 else codes
    eb = words_per_row(K if not transposed else rows) * (32 if form == q.QNN_FORM_I8 else 16)
    if not transposed:
        out = Guarded((rows, eb + 32), torch.uint8, fill=0x5C)
        q.qnn_quantize_form_kbit(dev(X), rows, K, K, bits, lo, hi, mode, form, out.t, eb + 32)
        want = _form_bytes_of(vals, K, form, q)
    else:
        # the same matrix read as [K' = rows, N' = K]: rows of the result run along the source's first index
        out = Guarded((K, eb + 32), torch.uint8, fill=0x5C)
        q.qnn_quantize_form_kbit_t(dev(X), rows, K, K, bits, lo, hi, mode, form, out.t, eb + 32)
        want = _form_bytes_of(vals.T, rows, form, q)
    torch.cuda.synchronize()
    got = out.t.cpu().numpy()
    np.testing.assert_array_equal(got[:, :eb], want)
    assert (got[:, eb:] == 0x5C).all()
    out.check()


def test_form_quantisers_feed_the_product(q):
    """fp32 -> form -> qnn_tc_gemm with no packed planes anywhere: the config-1 layer (100 x 4096 x 4096) against the oracle."""
    wl = workloads.fc_single()
    X, W = wl.X.numpy(), wl.W.numpy()
    M, K = X.shape
    N = W.shape[1]
    form = q.qnn_tc_form(1, q.QNN_MODE_PM1, 1, q.QNN_MODE_PM1, K)
    rb = q.qnn_tc_row_bytes(K, form)
    af = torch.empty(M, rb, dtype=torch.uint8, device="cuda")
    bf = torch.empty(N, rb, dtype=torch.uint8, device="cuda")
    q.qnn_quantize_form_sign(wl.X.cuda(), M, K, K, form, af, rb)
    q.qnn_quantize_form_sign_t(wl.W.cuda(), K, N, N, form, bf, rb)
    out = Guarded((M, N), torch.int32, fill=-7)
    q.qnn_tc_gemm(q.tc_operand(af, rb, form), q.tc_operand(bf, rb, form), M, N, K, out.t, N)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0
    np.testing.assert_array_equal(out.t.cpu().numpy(), oracle.xnor_gemm(X, W))
    out.check()


def test_form_quantiser_argument_errors(q):
    x = torch.zeros(4, 64, device="cuda")
    out = torch.zeros(4, 64, dtype=torch.uint8, device="cuda")
    with pytest.raises(q.QnnError) as e:
        q.qnn_quantize_form_kbit(x, 4, 64, 64, 4, -1.0, 1.0, 1, q.QNN_FORM_FP4, out, 64)      # 4-bit values do not fit e2m1
    assert e.value.status == q.QNN_ERR_UNSUPPORTED
    with pytest.raises(q.QnnError) as e:
        q.qnn_quantize_form_sign(x, 4, 64, 64, q.QNN_FORM_FP4, out, 24)                       # row stride not a multiple of 16
    assert e.value.status == q.QNN_ERR_ALIGNMENT
    with pytest.raises(q.QnnError) as e:
        q.qnn_quantize_form_sign(x, 4, 64, 64, 7, out, 64)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
