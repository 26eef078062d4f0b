"""GPU parity: XNOR and bit-plane matrix products (every algorithm the build offers) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_1609_07061_b200 import workloads
from util import Guarded, as_i32_words, dev, pack_bits_ref, unpack_words, words_np, words_per_row

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q():
    import paper_1609_07061_b200.binding as b
    return b


def _algos(q):
    return [q.QNN_ALGO_POPC, q.QNN_ALGO_B1_MMA, q.QNN_ALGO_TC_I8, q.QNN_ALGO_AUTO, q.QNN_ALGO_TC_FP4, q.QNN_ALGO_TC_PACKED]


def _ws(q, op, M, N, K, ka=1, kb=1, algo=0):
    n = q.qnn_workspace_bytes(op, M, N, K, ka, kb, algo)
    return torch.empty(max(n, 256), dtype=torch.uint8, device="cuda")


def _run_xnor(q, X, W, algo, lda_pad=0, ldo_pad=0):
    """X [M,K], W [K,N] float32 -> int32 [M,N] via test-side packing (independent of the GPU packers)."""
    M, K = X.shape
    N = W.shape[1]
    lda = words_per_row(K) + lda_pad
    a = pack_bits_ref((X >= 0).astype(np.uint8), lda)
    b = pack_bits_ref((W >= 0).astype(np.uint8).T, lda)
    out = Guarded((M, N + ldo_pad), torch.int32, fill=-7)
    ws = _ws(q, q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, algo)
    try:
        q.qnn_xnor_gemm(as_i32_words(a).cuda(), lda, as_i32_words(b).cuda(), lda, M, N, K, out.t, N + ldo_pad, algo, ws)
    except q.QnnError as e:
        if e.status == q.QNN_ERR_UNSUPPORTED:
            pytest.skip(f"algo {algo} does not support this shape: {e}")
        raise
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    out.check()
    res = out.t.cpu().numpy()
    if ldo_pad:
        assert (res[:, N:] == -7).all()
    return res[:, :N]


SHAPES = [(1, 1, 1), (2, 3, 31), (5, 7, 32), (3, 2, 33), (31, 33, 63), (32, 32, 64), (33, 31, 65), (63, 65, 127),
          (64, 64, 128), (65, 63, 129), (127, 129, 255), (129, 127, 257), (100, 10, 4096), (130, 300, 1000),
          (257, 513, 784), (1, 1000, 2304), (300, 1, 96)]


@pytest.mark.parametrize("algo_idx", [0, 1, 2, 3, 4])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_xnor_gemm_shapes(q, M, N, K, algo_idx):
    algo = _algos(q)[algo_idx]
    rng = np.random.default_rng(M * 100003 + N * 1009 + K)
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    got = _run_xnor(q, X, W, algo, lda_pad=(K % 3), ldo_pad=(N % 2))
    np.testing.assert_array_equal(got, oracle.xnor_gemm(X, W))


@pytest.mark.parametrize("algo_idx", [0, 1, 2, 3, 4])
def test_xnor_gemm_extremes(q, algo_idx):
    """All-agree, all-disagree and alternating rows: closed forms K, -K, 0."""
    algo = _algos(q)[algo_idx]
    K, N = 200, 40
    W = np.where(np.arange(K * N).reshape(K, N) % 3 == 0, 1.0, -1.0).astype(np.float32)
    X = np.stack([W[:, 5], -W[:, 5], np.ones(K, np.float32), -np.ones(K, np.float32)])
    got = _run_xnor(q, X, W, algo)
    assert got[0, 5] == K and got[1, 5] == -K
    np.testing.assert_array_equal(got, oracle.xnor_gemm(X, W))


@pytest.mark.parametrize("algo_idx", [0, 1, 2, 3, 4])
def test_fc_single_layer_config(q, algo_idx):
    """Config 1: X[100,4096] ~ N(0,1), W[4096,4096] ~ U(-1,1), seed 0, through the GPU packers and the product."""
    algo = _algos(q)[algo_idx]
    wl = workloads.fc_single()
    M, K = wl.X.shape
    N = wl.W.shape[1]
    ld = words_per_row(K)
    a = torch.zeros(M, ld, dtype=torch.int32, device="cuda")
    b = torch.zeros(N, ld, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_sign(wl.X.cuda(), M, K, K, a, ld)
    q.qnn_quantize_pack_sign_t(wl.W.cuda(), K, N, N, b, ld)
    out = Guarded((M, N), torch.int32, fill=-7)
    ws = _ws(q, q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, algo)
    try:
        q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, out.t, N, algo, ws)
    except q.QnnError as e:
        if e.status == q.QNN_ERR_UNSUPPORTED:
            pytest.skip(str(e))
        raise
    torch.cuda.synchronize()
    want = oracle.xnor_gemm(wl.X.numpy(), wl.W.numpy())
    np.testing.assert_array_equal(out.t.cpu().numpy(), want)
    out.check()
    # run-to-run determinism
    for _ in range(2):
        out2 = torch.empty(M, N, dtype=torch.int32, device="cuda")
        q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, out2, N, algo, ws)
        assert torch.equal(out2, out.t)


@pytest.mark.parametrize("algo_idx", [0, 1, 2, 3, 4])
@pytest.mark.parametrize("M,N,K", [(5, 7, 33), (64, 64, 128), (100, 130, 1000), (257, 96, 784), (33, 4096, 96)])
@pytest.mark.parametrize("with_flip", [False, True])
def test_xnor_gemm_threshold(q, M, N, K, with_flip, algo_idx):
    algo = _algos(q)[algo_idx]
    rng = np.random.default_rng(M + N + K)
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    s = oracle.xnor_gemm(X, W)
    T = rng.integers(-20, 21, N).astype(np.int32)
    T[::4] = s[0, ::4]                                   # exact equalities on row 0
    flip = rng.integers(0, 2, N).astype(np.uint8) if with_flip else None
    lda = words_per_row(K)
    a = pack_bits_ref((X >= 0).astype(np.uint8), lda)
    b = pack_bits_ref((W >= 0).astype(np.uint8).T, lda)
    ldb = words_per_row(N) + 1
    out = Guarded((M, ldb), torch.int32, fill=0x77777777)
    ws = _ws(q, q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, algo)
    try:
        q.qnn_xnor_gemm_threshold(as_i32_words(a).cuda(), lda, as_i32_words(b).cuda(), lda, M, N, K, dev(T),
                                  None if flip is None else dev(flip), out.t, ldb, algo, ws)
    except q.QnnError as e:
        if e.status == q.QNN_ERR_UNSUPPORTED:
            pytest.skip(str(e))
        raise
    torch.cuda.synchronize()
    np.testing.assert_array_equal(unpack_words(words_np(out.t), N), oracle.threshold(s, T, flip))
    assert (words_np(out.t)[:, words_per_row(N):] == 0x77777777).all()
    out.check()


def _planes_ref(codes, bits, ld):
    """codes [rows,K] -> uint32 [bits, rows, ld] (test-side packing)."""
    return np.stack([pack_bits_ref(((codes >> i) & 1).astype(np.uint8), ld) for i in range(bits)])


def _values(codes, bits, mode):
    return codes.astype(np.int32) if mode == 0 else (2 * codes.astype(np.int32) - ((1 << bits) - 1))


@pytest.mark.parametrize("algo_idx", [0, 2, 3, 4])
@pytest.mark.parametrize("ka,a_mode,kb,b_mode", [(8, 0, 1, 1), (2, 0, 1, 1), (4, 1, 4, 1), (1, 1, 1, 1), (3, 0, 2, 0),
                                                 (2, 1, 3, 0), (1, 0, 1, 0), (8, 0, 8, 0), (7, 1, 7, 1), (8, 1, 2, 1)])
@pytest.mark.parametrize("M,N,K", [(3, 5, 31), (65, 33, 100), (130, 257, 800)])
def test_bitplane_gemm_modes(q, ka, a_mode, kb, b_mode, M, N, K, algo_idx):
    algo = _algos(q)[algo_idx]
    rng = np.random.default_rng(ka * 1000 + kb * 100 + M + N + K + a_mode * 7 + b_mode * 3)
    qa = rng.integers(0, 1 << ka, (M, K)).astype(np.int32)
    qb = rng.integers(0, 1 << kb, (K, N)).astype(np.int32)
    ld = words_per_row(K) + 1
    ap = _planes_ref(qa, ka, ld)
    bp = _planes_ref(qb.T, kb, ld)
    out = Guarded((M, N), torch.int32, fill=-7)
    ws = _ws(q, q.QNN_OP_BITPLANE_GEMM, M, N, K, ka, kb, algo)
    try:
        q.qnn_bitplane_gemm(as_i32_words(ap).cuda(), ka, a_mode, ld, M * ld, as_i32_words(bp).cuda(), kb, b_mode, ld,
                            N * ld, M, N, K, out.t, N, algo, ws)
    except q.QnnError as e:
        if e.status == q.QNN_ERR_UNSUPPORTED:
            pytest.skip(str(e))
        raise
    torch.cuda.synchronize()
    want = oracle.int_gemm(_values(qa, ka, a_mode), _values(qb, kb, b_mode))
    np.testing.assert_array_equal(out.t.cpu().numpy(), want)
    out.check()


@pytest.mark.parametrize("algo_idx", [0, 2, 3, 4])
def test_bitplane_gemm_threshold(q, algo_idx):
    algo = _algos(q)[algo_idx]
    rng = np.random.default_rng(99)
    M, N, K, ka = 70, 200, 784, 8
    qa = rng.integers(0, 256, (M, K)).astype(np.int32)
    wb = np.where(rng.uniform(-1, 1, (K, N)) >= 0, 1, 0).astype(np.int32)
    ld = 28
    ap = _planes_ref(qa, ka, ld)
    bp = _planes_ref(wb.T, 1, ld)
    s = oracle.int_gemm(qa, 2 * wb - 1)
    T = rng.integers(-3000, 3000, N).astype(np.int32)
    T[::5] = s[3, ::5]
    flip = rng.integers(0, 2, N).astype(np.uint8)
    out = Guarded((M, 7), torch.int32, fill=0)
    ws = _ws(q, q.QNN_OP_BITPLANE_GEMM, M, N, K, ka, 1, algo)
    try:
        q.qnn_bitplane_gemm_threshold(as_i32_words(ap).cuda(), ka, 0, ld, M * ld, as_i32_words(bp).cuda(), 1, 1, ld, 0,
                                      M, N, K, dev(T), dev(flip), out.t, 7, algo, ws)
    except q.QnnError as e:
        if e.status == q.QNN_ERR_UNSUPPORTED:
            pytest.skip(str(e))
        raise
    torch.cuda.synchronize()
    np.testing.assert_array_equal(unpack_words(words_np(out.t), N), oracle.threshold(s, T, flip))
    out.check()


def test_padding_invariance(q):
    """K = 784 padded to 800, 1024 (zero pad bits in both operands) gives the same product."""
    rng = np.random.default_rng(784)
    M, N, K = 40, 50, 784
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    want = oracle.xnor_gemm(X, W)
    for ld in (25, 28, 32):
        a = pack_bits_ref((X >= 0).astype(np.uint8), ld)
        b = pack_bits_ref((W >= 0).astype(np.uint8).T, ld)
        out = torch.empty(M, N, dtype=torch.int32, device="cuda")
        q.qnn_xnor_gemm(as_i32_words(a).cuda(), ld, as_i32_words(b).cuda(), ld, M, N, K, out, N, q.QNN_ALGO_POPC)
        np.testing.assert_array_equal(out.cpu().numpy(), want)


# ---- QNN_ALGO_TC_PACKED: the tensor-core product straight from packed tiles (no workspace) ---------------------------

def _ld4(K):
    return (words_per_row(K) + 3) // 4 * 4          # rows TMA can address: a multiple of 16 bytes apart


@pytest.mark.parametrize("ka,a_mode,kb,b_mode", [(1, 1, 1, 1), (2, 0, 1, 1), (2, 1, 1, 1), (1, 0, 1, 1), (2, 0, 2, 1), (1, 1, 2, 0)])
@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (5, 7, 31), (100, 130, 1000), (128, 32, 256), (129, 33, 257), (300, 70, 2048), (37, 257, 2049),
                                   (64, 96, 4500)])
def test_tc_packed_bitplane_products(q, ka, a_mode, kb, b_mode, M, N, K):
    """Packed planes in, int32 out, nothing in between: ragged M / N / K, several row tiles, more than one packed tile along
    K (2048 elements each), one- and two-plane operands in both value modes; every output against the oracle."""
    rng = np.random.default_rng(ka * 100 + kb * 10 + a_mode + M + N + K)
    qa = rng.integers(0, 1 << ka, (M, K)).astype(np.int32)
    qb = rng.integers(0, 1 << kb, (K, N)).astype(np.int32)
    ld = _ld4(K) + 4
    ap = _planes_ref(qa, ka, ld)
    bp = _planes_ref(qb.T, kb, ld)
    out = Guarded((M, N + 1), torch.int32, fill=-7)
    q.qnn_bitplane_gemm(as_i32_words(ap).cuda(), ka, a_mode, ld, M * ld, as_i32_words(bp).cuda(), kb, b_mode, ld, N * ld, M, N, K,
                        out.t, N + 1, q.QNN_ALGO_TC_PACKED, None)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    got = out.t.cpu().numpy()
    np.testing.assert_array_equal(got[:, :N], oracle.int_gemm(_values(qa, ka, a_mode), _values(qb, kb, b_mode)))
    assert (got[:, N:] == -7).all()
    out.check()


@pytest.mark.parametrize("M,N,K", [(100, 4096, 4096), (130, 300, 1000), (3, 40, 96)])
def test_tc_packed_threshold_bits(q, M, N, K):
    """Thresholded bits out of the packed-tile kernel, with exact equalities planted and flips."""
    rng = np.random.default_rng(M + N + K)
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    s = oracle.xnor_gemm(X, W)
    T = rng.integers(-40, 41, N).astype(np.int32)
    T[::3] = s[M // 2, ::3]
    flip = rng.integers(0, 2, N).astype(np.uint8)
    ld = _ld4(K)
    a = as_i32_words(pack_bits_ref((X >= 0).astype(np.uint8), ld)).cuda()
    b = as_i32_words(pack_bits_ref((W >= 0).astype(np.uint8).T, ld)).cuda()
    ldw = words_per_row(N) + 1
    bits = Guarded((M, ldw), torch.int32, fill=0x77777777)
    q.qnn_xnor_gemm_threshold(a, ld, b, ld, M, N, K, dev(T), dev(flip), bits.t, ldw, q.QNN_ALGO_TC_PACKED, None)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    np.testing.assert_array_equal(unpack_words(words_np(bits.t), N), oracle.threshold(s, T, flip))
    assert (words_np(bits.t)[:, words_per_row(N):] == 0x77777777).all()
    bits.check()


def test_tc_packed_refuses_what_it_cannot_run(q):
    fake = torch.zeros(4096, dtype=torch.int32, device="cuda")
    out = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(q.QnnError) as e:           # rows 20 bytes apart: not addressable by TMA
        q.qnn_xnor_gemm(fake, 5, fake, 5, 8, 8, 160, out, 8, q.QNN_ALGO_TC_PACKED, None)
    assert e.value.status == q.QNN_ERR_UNSUPPORTED
    with pytest.raises(q.QnnError) as e:           # 4 planes do not fit e2m1
        q.qnn_bitplane_gemm(fake, 4, 1, 8, 64, fake, 1, 1, 8, 0, 8, 8, 256, out, 8, q.QNN_ALGO_TC_PACKED, None)
    assert e.value.status == q.QNN_ERR_UNSUPPORTED


def test_auto_without_workspace_stays_on_the_tensor_cores_for_small_batches(q):
    """QNN_ALGO_AUTO with no workspace: small batches take the packed-tile kernel (and say so), bit-exact."""
    wl = workloads.fc_single()
    X, W = wl.X.numpy(), wl.W.numpy()
    M, K = X.shape
    N = W.shape[1]
    ld = K // 32
    a = as_i32_words(pack_bits_ref((X >= 0).astype(np.uint8), ld)).cuda()
    b = as_i32_words(pack_bits_ref((W >= 0).astype(np.uint8).T, ld)).cuda()
    out = Guarded((M, N), torch.int32, fill=-7)
    before = q.qnn_launch_count()
    q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, out.t, N, q.QNN_ALGO_AUTO, None)
    assert q.qnn_launch_count() == before + 1          # one launch, nothing rewritten
    assert "packed tiles" in q.qnn_last_error()
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0
    np.testing.assert_array_equal(out.t.cpu().numpy(), oracle.xnor_gemm(X, W))
    out.check()
