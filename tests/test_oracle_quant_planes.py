"""Pins for the k-bit linear quantiser (Eq. 9), bit-planes and the bit-plane product (Eq. 8)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_1609_07061_b200 import workloads


def _read(golden_dir, name):
    with open(os.path.join(golden_dir, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_linear_quant_golden(golden_dir):
    rows = _read(golden_dir, "linear_quant_2bit.txt")
    x = np.array([float(r[0]) for r in rows], np.float32)
    want = np.array([int(r[1]) for r in rows], np.int32)
    np.testing.assert_array_equal(oracle.linear_quant_codes(x, 2, 0.0, 1.0), want)


@pytest.mark.parametrize("bits", [1, 2, 4, 8])
@pytest.mark.parametrize("lo,hi", [(0.0, 1.0), (-1.0, 1.0), (-3.0, 5.0)])
def test_level_centres_are_fixed_points(bits, lo, hi):
    L = (1 << bits) - 1
    q = np.arange(L + 1)
    centres = (lo + q.astype(np.float64) * (hi - lo) / L).astype(np.float32)
    np.testing.assert_array_equal(oracle.linear_quant_codes(centres, bits, lo, hi), q)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_monotone_clipped_and_bounded(bits):
    x = np.linspace(-2.0, 2.0, 20001).astype(np.float32)
    q = oracle.linear_quant_codes(x, bits, -1.0, 1.0)
    assert np.all(np.diff(q) >= 0)
    assert q.min() == 0 and q.max() == (1 << bits) - 1
    assert np.all(q[x <= -1.0] == 0) and np.all(q[x >= 1.0] == (1 << bits) - 1)
    assert len(np.unique(q)) == 1 << bits


def test_ties_go_to_even():
    # lo=0, hi=15 with 4 bits makes the step exactly 1, so j+0.5 is an exact tie
    x = np.arange(0, 15, dtype=np.float32) + 0.5
    q = oracle.linear_quant_codes(x, 4, 0.0, 15.0)
    want = np.array([0, 2, 2, 4, 4, 6, 6, 8, 8, 10, 10, 12, 12, 14, 14], np.int32)
    np.testing.assert_array_equal(q, want)


@pytest.mark.parametrize("bits,lo,hi", [(2, 0.0, 1.0), (4, -1.0, 1.0), (8, 0.0, 1.0)])
def test_against_torch_round_on_same_quotient(bits, lo, hi):
    """torch.round is also round-half-to-even: an independent library witness on the same fp32 steps."""
    g = torch.Generator().manual_seed(11)
    x = (torch.randn(50000, generator=g) * 0.8).to(torch.float32)
    inv = torch.tensor(float(oracle.inv_step(bits, lo, hi)), dtype=torch.float32)
    t = torch.clamp(x, lo, hi)
    u = (t - torch.tensor(lo, dtype=torch.float32)) * inv
    want = torch.round(u).to(torch.int32).clamp(0, (1 << bits) - 1).numpy()
    np.testing.assert_array_equal(oracle.linear_quant_codes(x.numpy(), bits, lo, hi), want)


def test_nan_and_infinities():
    x = np.array([np.nan, np.inf, -np.inf], np.float32)
    np.testing.assert_array_equal(oracle.linear_quant_codes(x, 4, -1.0, 1.0), [0, 15, 0])


@pytest.mark.parametrize("bits", [1, 2, 4, 8])
def test_bit_plane_reconstruction(bits):
    q = np.arange(1 << bits, dtype=np.int32)
    rec = sum((1 << i) * oracle.bit_plane(q, i).astype(np.int64) for i in range(bits))
    np.testing.assert_array_equal(rec, q)
    # symmetric reading: 2q - (2^k - 1) = sum_i 2^i s_i, s_i = +-1 from bit i
    sym = sum((1 << i) * (2 * oracle.bit_plane(q, i).astype(np.int64) - 1) for i in range(bits))
    np.testing.assert_array_equal(oracle.codes_to_symmetric(q, bits), sym)


def test_eq8_golden(golden_dir):
    rows = _read(golden_dir, "eq8_bitplanes.txt")
    x = np.array([[int(v) for v in r[1:]] for r in rows if r[0] == "x"], np.int32)
    w = np.array([[int(v) for v in r[1:]] for r in rows if r[0] == "w"], np.int32).T
    s = int([r for r in rows if r[0] == "s"][0][1])
    for r in rows:
        if r[0] == "plane":
            n = int(r[1])
            np.testing.assert_array_equal(oracle.bit_plane(x[0], n - 1), [int(v) for v in r[2:5]])
            dot = oracle.int_gemm(oracle.bit_plane(x, n - 1).astype(np.int32), w)
            assert int(dot[0, 0]) == int(r[5])
    assert int(oracle.int_gemm(x, w)[0, 0]) == s
    assert int(oracle.planewise_gemm(x, 8, w)[0, 0]) == s


@pytest.mark.parametrize("M,N,K,ka", [(3, 4, 5, 8), (7, 3, 33, 2), (2, 9, 100, 4)])
def test_planewise_equals_integer_product_and_float64(M, N, K, ka):
    rng = np.random.default_rng(M + N + K)
    Q = rng.integers(0, 1 << ka, (M, K)).astype(np.int32)
    B = np.where(rng.uniform(-1, 1, (K, N)) >= 0, 1, -1).astype(np.int32)
    got = oracle.int_gemm(Q, B)
    np.testing.assert_array_equal(got, oracle.planewise_gemm(Q, ka, B))
    np.testing.assert_array_equal(got, (Q.astype(np.float64) @ B.astype(np.float64)).astype(np.int32))


def test_one_bit_symmetric_case_reduces_to_xnor():
    rng = np.random.default_rng(5)
    X = rng.standard_normal((6, 70)).astype(np.float32)
    W = rng.standard_normal((70, 5)).astype(np.float32)
    qa = oracle.linear_quant_codes(np.where(X >= 0, 1.0, -1.0), 1, -1.0, 1.0)
    qb = oracle.linear_quant_codes(np.where(W >= 0, 1.0, -1.0), 1, -1.0, 1.0)
    got = oracle.int_gemm(oracle.codes_to_symmetric(qa, 1), oracle.codes_to_symmetric(qb, 1))
    np.testing.assert_array_equal(got, oracle.xnor_gemm(X, W))


def test_lstm_levels_roundtrip_and_real_product():
    wl = workloads.lstm_gate(M=9, K=64, N=7, seed=4)
    qa = oracle.linear_quant_codes(wl.X.numpy(), 4, -1.0, 1.0)
    qb = oracle.linear_quant_codes(wl.W.numpy(), 4, -1.0, 1.0)
    va = oracle.codes_to_symmetric(qa, 4)
    vb = oracle.codes_to_symmetric(qb, 4)
    # the generator's real values are exactly v/15
    np.testing.assert_allclose(va / 15.0, wl.X.numpy().astype(np.float64), atol=1e-6)
    got = oracle.int_gemm(va, vb)
    real = wl.X.numpy().astype(np.float64) @ wl.W.numpy().astype(np.float64)
    np.testing.assert_allclose(got / 225.0, real, atol=1e-4)


def test_ap2_exponent_pins():
    """AP2(x) = sign(x) 2^round(log2|x|): float64 logarithms away from ties, closed forms at and around them."""
    rng = np.random.default_rng(7)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    x = x[x != 0]
    l2 = np.log2(np.abs(x.astype(np.float64)))
    far = np.abs(l2 - np.floor(l2) - 0.5) > 1e-6               # a float64 log cannot be trusted to decide a near tie
    e = oracle.ap2_exponent(x)
    np.testing.assert_array_equal(e[far], np.round(l2[far]).astype(np.int32))
    # the chosen power of two is within a factor sqrt(2) of |x|, on every input
    ratio = np.abs(x.astype(np.float64)) / np.exp2(e.astype(np.float64))
    assert np.all(ratio > 2 ** -0.5) and np.all(ratio < 2 ** 0.5)
    # powers of two are fixed points; sign does not matter
    p = np.array([2.0 ** k for k in range(-30, 31)], np.float32)
    np.testing.assert_array_equal(oracle.ap2_exponent(p), np.arange(-30, 31))
    np.testing.assert_array_equal(oracle.ap2_exponent(-p), np.arange(-30, 31))
    # the two floats around sqrt(2): the one below rounds down, the one above rounds up (at every scale)
    lo = np.float32(1.41421353816986083984375)
    hi = np.nextafter(lo, np.float32(2.0))
    assert float(lo) ** 2 < 2.0 < float(hi) ** 2
    for k in (-5, 0, 9):
        s = np.float32(2.0 ** k)
        np.testing.assert_array_equal(oracle.ap2_exponent(np.array([lo * s, hi * s], np.float32)), [k, k + 1])
    # 1.5 has log2 = 0.585 -> 1;  1.25 -> 0;  3 -> 2 (log2 3 = 1.585);  denormals have exponents below -126
    np.testing.assert_array_equal(oracle.ap2_exponent(np.array([1.5, 1.25, 3.0, 0.75], np.float32)), [1, 0, 2, 0])
    assert oracle.ap2_exponent(np.array([1e-40], np.float32))[0] < -126
    # monotone in |x|
    xs = np.sort(np.abs(x))
    assert np.all(np.diff(oracle.ap2_exponent(xs)) >= 0)
    sp = oracle.ap2_exponent(np.array([0.0, -0.0, np.inf, -np.inf, np.nan], np.float32))
    assert sp[0] == sp[1] == np.iinfo(np.int32).min and sp[2] == sp[3] == sp[4] == np.iinfo(np.int32).max


def test_log_quant_pins():
    """Eq. 10: magnitudes clip to [2^emin, 2^emax]; result in units of 2^emin, sign of Eq. 1."""
    x = np.array([0.0, -0.0, 1e-9, -1e-9, 0.24, 0.26, -0.7, 0.71, 1.0, -1.4, 1.42, 3.0, 100.0, -100.0, np.inf, -np.inf, np.nan],
                 np.float32)
    v = oracle.log_quant(x, -2, 1)               # levels 1/4, 1/2, 1, 2  ->  1, 2, 4, 8
    np.testing.assert_array_equal(v, [1, 1, 1, -1, 1, 1, -2, 4, 4, -4, 8, 8, 8, -8, 8, -8, -8])
    # agreement with the literal formula in float64 on random data away from ties
    rng = np.random.default_rng(3)
    y = (rng.standard_normal(5000) * 2.0).astype(np.float32)
    y = y[y != 0]
    l2 = np.log2(np.abs(y.astype(np.float64)))
    far = np.abs(l2 - np.floor(l2) - 0.5) > 1e-6
    want = np.where(y >= 0, 1, -1) * np.exp2(np.clip(np.round(l2), -3, 3) + 3)
    np.testing.assert_array_equal(oracle.log_quant(y, -3, 3)[far], want[far].astype(np.int32))
    # at most (emax - emin + 1) magnitudes, all powers of two
    mags = np.unique(np.abs(oracle.log_quant(y, -3, 3)))
    assert set(mags.tolist()) <= {1, 2, 4, 8, 16, 32, 64}
    with pytest.raises(ValueError):
        oracle.log_quant(y, 2, 1)


def test_log_gemm_pins():
    """Algorithm 1's backward products on Eq. 10 codes: out = sum_k sign(x) 2^clamp(round(log2|x|)) w, in units of 2^emin."""
    from fractions import Fraction
    import math
    rng = np.random.default_rng(11)
    # (i) exact rational arithmetic on inputs away from the rounding ties
    M, K, N, emin, emax = 5, 23, 4, -12, 3
    x = (rng.standard_normal((M, K)) * np.exp2(rng.integers(-14, 5, (M, K)))).astype(np.float32)
    l2 = np.log2(np.abs(x.astype(np.float64)))
    assert np.all(np.abs(l2 - np.floor(l2) - 0.5) > 1e-6)
    w = rng.integers(0, 2, (K, N)) * 2 - 1
    got = oracle.log_gemm(x, w, emin, emax)
    assert got.dtype == np.int64
    for m in range(M):
        for n in range(N):
            acc = Fraction(0)
            for k in range(K):
                e = min(max(round(math.log2(abs(float(x[m, k])))), emin), emax)
                acc += (1 if x[m, k] >= 0 else -1) * Fraction(2) ** e * int(w[k, n])
            assert Fraction(int(got[m, n])) * Fraction(2) ** emin == acc
    # (ii) constant rows: every element 2^e0 gives 2^(e0 - emin) * sum(w); clipping at both ends
    ones = np.full((2, K), 0.25, np.float32)
    np.testing.assert_array_equal(oracle.log_gemm(ones, w, -4, 2), np.tile(4 * w.sum(axis=0), (2, 1)))
    tiny, huge = np.full((1, K), 1e-30, np.float32), np.full((1, K), -1e30, np.float32)
    np.testing.assert_array_equal(oracle.log_gemm(tiny, w, -4, 2), w.sum(axis=0)[None, :])
    np.testing.assert_array_equal(oracle.log_gemm(huge, w, -4, 2), -64 * w.sum(axis=0)[None, :])
    # (iii) the full 31-exponent range of a 6-bit code: sums beyond int32 stay exact
    big = np.full((1, 8), 1.0, np.float32)
    np.testing.assert_array_equal(oracle.log_gemm(big, np.ones((8, 1), np.int64), -30, 0), [[8 * 2 ** 30]])
    mixed = np.array([[1.0, 2.0 ** -30, -(2.0 ** -15)]], np.float32)
    np.testing.assert_array_equal(oracle.log_gemm(mixed, np.array([[1], [1], [1]]), -30, 0), [[2 ** 30 + 1 - 2 ** 15]])
    # (iv) additivity in w, oddness in x
    w2 = rng.integers(-3, 4, (K, N))
    np.testing.assert_array_equal(oracle.log_gemm(x, w + w2, emin, emax), oracle.log_gemm(x, w, emin, emax) + oracle.log_gemm(x, w2, emin, emax))
    nz = np.where(x == 0, np.float32(1.0), x)
    np.testing.assert_array_equal(oracle.log_gemm(-nz, w, emin, emax), -oracle.log_gemm(nz, w, emin, emax))
    with pytest.raises(ValueError):
        oracle.log_gemm(x, w, -31, 0)
