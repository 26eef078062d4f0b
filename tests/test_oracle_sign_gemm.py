"""Pins for the oracle's sign and +-1 matrix product (Eq. 1, Algorithm 4, Eq. 11).

None of these tests re-types the oracle's own loop: they compare it with
hand-computed fixtures, brute-force float64 dot products, a library matmul,
an independent word-level popcount identity, and closed forms.
"""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_1609_07061_b200 import workloads


def _read(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_sign_golden(golden_dir):
    rows = _read(golden_dir, "sign_eq1.txt")
    x = np.array([float(r[0]) for r in rows], np.float32)
    want = np.array([int(r[1]) for r in rows], np.int32)
    np.testing.assert_array_equal(oracle.sign(x), want)


def test_sign_negative_zero_is_plus_one():
    x = np.array([0.0, -0.0], np.float32)
    assert np.signbit(x[1])
    np.testing.assert_array_equal(oracle.sign(x), [1, 1])


def test_xnor_gemm_golden(golden_dir):
    rows = _read(golden_dir, "xnor_dot_small.txt")
    X = np.array([[float(v) for v in r[1:]] for r in rows if r[0] == "X"], np.float32)
    W = np.array([[float(v) for v in r[1:]] for r in rows if r[0] == "W"], np.float32)
    Y = np.array([[int(v) for v in r[1:]] for r in rows if r[0] == "Y"], np.int32)
    np.testing.assert_array_equal(oracle.xnor_gemm(X, W), Y)


@pytest.mark.parametrize("K", [1, 2, 3, 4])
def test_xnor_gemm_exhaustive_tiny(K):
    """Every pair of +-1 vectors of length K, against a float64 dot product."""
    vecs = np.array(list(itertools.product([-1.0, 1.0], repeat=K)), np.float64)   # [2^K, K]
    X = (vecs * 0.37).astype(np.float32)           # magnitudes are irrelevant, only the sign
    W = (vecs.T * 2.5).astype(np.float32)          # [K, 2^K]
    got = oracle.xnor_gemm(X, W)
    want = vecs @ vecs.T
    np.testing.assert_array_equal(got, want.astype(np.int32))


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (3, 5, 7), (17, 9, 33), (8, 31, 64), (5, 2, 257)])
def test_xnor_gemm_vs_library_matmul(M, N, K):
    """The float kernel and the XNOR kernel agree on +-1 inputs (Section 6): float64 matmul witness."""
    rng = np.random.default_rng(M * 1000 + N * 10 + K)
    X = rng.standard_normal((M, K)).astype(np.float32)
    W = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    sx = np.where(X >= 0, 1.0, -1.0)
    sw = np.where(W >= 0, 1.0, -1.0)
    np.testing.assert_array_equal(oracle.xnor_gemm(X, W), (sx @ sw).astype(np.int32))


def _pack_words_py(bits01):
    """Independent packer for the test: Python ints, element k -> bit k%32 of word k//32."""
    words = []
    for w0 in range(0, len(bits01), 32):
        v = 0
        for j, b in enumerate(bits01[w0:w0 + 32]):
            v |= int(b) << j
        words.append(v)
    return words


@pytest.mark.parametrize("K", [1, 31, 32, 33, 65, 784])
def test_popcount_identity(K):
    """dot = K - 2*popc(a xor b) over words whose pad bits are zero in BOTH operands (Eq. 11 reading)."""
    rng = np.random.default_rng(K)
    x = rng.standard_normal((4, K)).astype(np.float32)
    w = rng.standard_normal((K, 3)).astype(np.float32)
    got = oracle.xnor_gemm(x, w)
    for m in range(4):
        for n in range(3):
            a = _pack_words_py(x[m] >= 0)
            b = _pack_words_py(w[:, n] >= 0)
            pc = sum(bin(ai ^ bi).count("1") for ai, bi in zip(a, b))
            assert got[m, n] == K - 2 * pc
            # a pad bit set in only one operand breaks the identity (negative control)
            if K % 32:
                a_bad = list(a)
                a_bad[-1] |= 1 << (K % 32)
                pc_bad = sum(bin(ai ^ bi).count("1") for ai, bi in zip(a_bad, b))
                assert K - 2 * pc_bad != got[m, n]


def test_closed_forms():
    rng = np.random.default_rng(7)
    K, N = 129, 6
    W = rng.uniform(-1, 1, (K, N)).astype(np.float32)
    sw = np.where(W >= 0, 1, -1)
    # a row equal to a weight column gives K, its negation gives -K
    X = np.stack([W[:, 2], -W[:, 2] - 1e-9, np.ones(K, np.float32)]).astype(np.float32)
    X[1] = np.where(sw[:, 2] > 0, -1.0, 1.0)
    Y = oracle.xnor_gemm(X, W)
    assert Y[0, 2] == K and Y[1, 2] == -K
    np.testing.assert_array_equal(Y[2], sw.sum(axis=0))          # all +1 row -> column sums
    assert np.all(np.abs(Y) <= K)
    assert np.all((Y - K) % 2 == 0)                               # dot has the parity of K


def test_asymmetric_operands_not_transposed():
    """A [2,3]x[3,4] case whose transposed/misindexed variants give different answers."""
    X = np.array([[1, -1, 1], [-1, -1, 1]], np.float32)
    W = np.array([[1, 1, -1, -1], [1, -1, 1, -1], [-1, -1, -1, 1]], np.float32)
    want = np.array([[-1, 1, -3, 1], [-3, -1, -1, 3]], np.int32)    # by hand
    np.testing.assert_array_equal(oracle.xnor_gemm(X, W), want)


def test_statistics_on_seeded_layer():
    wl = workloads.fc_single(M=16, K=4096, N=512, seed=0)
    Y = oracle.xnor_gemm(wl.X.numpy(), wl.W.numpy()).astype(np.float64)
    assert abs(Y.mean()) < 3.0
    assert 0.8 * 4096 < Y.var() < 1.2 * 4096


def test_int_gemm_overflow_detected():
    A = np.full((1, 4), 2**30, np.int32)
    B = np.full((4, 1), 4, np.int32)
    with pytest.raises(OverflowError):
        oracle.int_gemm(A, B)
