"""CPU oracle for the quantised-network forward path -- TEST INFRASTRUCTURE.

A thin numpy/ctypes front for ``qnn_oracle.c`` (plain scalar C on unpacked
values, written from the paper's definitions).  It is independent of the CUDA
library: nothing here imports the product package, and the product package never
imports this.  Only the tests, the smoke check and the benchmark's CPU baseline
use it.

Pins (what each routine is checked against, other than itself) live in
``tests/test_oracle_*.py``:
  sign            Eq. 1 boundary values (+0, -0, denormals, inf, NaN)
  xnor_gemm       float64 dot products of sign values, exhaustive tiny K,
                  a library float64 matmul, closed forms, parity and bounds
  linear_quant    level centres, monotonicity, clipping, ties-to-even,
                  torch.round on the same fp32 quotient
  int_gemm        Eq. 8 evaluated plane by plane, float64 matmul on codes
  threshold       brute force; the batch-norm fold against direct double BN
  conv2d          library conv2d in float64 on +-1 tensors padded with +1,
                  the 1x1 case against the matrix product, all-ones input
  mlp_forward     Algorithm 4 step by step with the routines above
  ap2 / log_quant float64 round(log2|x|) away from ties, exact powers of two, the factor-sqrt(2)
                  bound, monotonicity, clipping, zero / infinities / NaN
  log_gemm        exact rational arithmetic (fractions) on small inputs built from the literal
                  sign * 2^round(log2|x|), closed forms (constant rows, clipping at both ends, the
                  31-exponent range beyond int32), additivity in w
  maxpool2x2      library max_pool2d in float64; the identity that pooling the
                  integer sums and then thresholding equals OR (AND where the
                  comparison is flipped) of the thresholded bits, by brute force
  convnet_forward Table 7 layer by layer against a float64 library chain
                  (conv2d, max_pool2d, comparisons)
  rescale         float64 numpy expression
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qnn_oracle.c")
_LIB = os.path.join(_HERE, "libqnn_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-std=c11", "-Wall", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.qo_num_threads.restype = ctypes.c_int
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=dtype)


def _check(rc: int, what: str) -> None:
    if rc == 1:
        raise OverflowError(f"oracle {what}: a result does not fit int32")
    if rc != 0:
        raise ValueError(f"oracle {what}: invalid argument (code {rc})")


def num_threads() -> int:
    return int(_load().qo_num_threads())


def sign(x) -> np.ndarray:
    """Eq. 1: +1 where x >= 0, else -1 (int32)."""
    x = _c(x, np.float32)
    out = np.empty(x.shape, np.int32)
    _check(_load().qo_sign(_ptr(x), ctypes.c_int64(x.size), _ptr(out)), "sign")
    return out


def inv_step(bits: int, lo: float, hi: float) -> np.float32:
    """(2^bits - 1) / (hi - lo) in fp32, the constant both implementations share."""
    return np.float32(np.float32((1 << bits) - 1) / (np.float32(hi) - np.float32(lo)))


def linear_quant_codes(x, bits: int, lo: float, hi: float) -> np.ndarray:
    """Eq. 9 as a uniform quantiser: integer code in [0, 2^bits - 1]."""
    x = _c(x, np.float32)
    q = np.empty(x.shape, np.int32)
    rc = _load().qo_linear_quant_codes(_ptr(x), ctypes.c_int64(x.size), ctypes.c_int(bits),
                                       ctypes.c_float(lo), ctypes.c_float(hi),
                                       ctypes.c_float(float(inv_step(bits, lo, hi))), _ptr(q))
    _check(rc, "linear_quant_codes")
    return q


def codes_to_symmetric(q, bits: int) -> np.ndarray:
    q = _c(q, np.int32)
    v = np.empty(q.shape, np.int32)
    _check(_load().qo_codes_to_symmetric(_ptr(q), ctypes.c_int64(q.size), ctypes.c_int(bits), _ptr(v)),
           "codes_to_symmetric")
    return v


def bit_plane(q, i: int) -> np.ndarray:
    """Plane i (0 = least significant) of non-negative integer codes, as uint8 0/1."""
    q = _c(q, np.int32)
    p = np.empty(q.shape, np.uint8)
    _check(_load().qo_bit_plane(_ptr(q), ctypes.c_int64(q.size), ctypes.c_int(i), _ptr(p)), "bit_plane")
    return p


def int_gemm(A, B) -> np.ndarray:
    """out[m,n] = sum_k A[m,k] * B[k,n] on int32 values, exact."""
    A = _c(A, np.int32)
    B = _c(B, np.int32)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    out = np.empty((M, N), np.int32)
    rc = _load().qo_int_gemm(_ptr(A), _ptr(B), ctypes.c_int64(M), ctypes.c_int64(N), ctypes.c_int64(K),
                             _ptr(out))
    _check(rc, "int_gemm")
    return out


def xnor_gemm(X, W) -> np.ndarray:
    """Y[m,n] = sum_k sign(X[m,k]) * sign(W[k,n]); X [M,K], W [K,N] fp32."""
    X = _c(X, np.float32)
    W = _c(W, np.float32)
    M, K = X.shape
    K2, N = W.shape
    assert K == K2
    out = np.empty((M, N), np.int32)
    rc = _load().qo_xnor_gemm(_ptr(X), _ptr(W), ctypes.c_int64(M), ctypes.c_int64(N), ctypes.c_int64(K),
                              _ptr(out))
    _check(rc, "xnor_gemm")
    return out


def planewise_gemm(QA, ka: int, B) -> np.ndarray:
    """Eq. 8 literally: sum_i 2^i * (plane_i(QA) . B)."""
    QA = _c(QA, np.int32)
    B = _c(B, np.int32)
    M, K = QA.shape
    K2, N = B.shape
    assert K == K2
    out = np.empty((M, N), np.int32)
    rc = _load().qo_planewise_gemm(_ptr(QA), ctypes.c_int(ka), _ptr(B), ctypes.c_int64(M),
                                   ctypes.c_int64(N), ctypes.c_int64(K), _ptr(out))
    _check(rc, "planewise_gemm")
    return out


def threshold(s, T, flip=None) -> np.ndarray:
    """bit[m,n] = (s[m,n] >= T[n]) xor flip[n], one uint8 per element."""
    s = _c(s, np.int32)
    M, N = s.shape
    T = _c(T, np.int32)
    assert T.shape == (N,)
    f = None if flip is None else _c(flip, np.uint8)
    bits = np.empty((M, N), np.uint8)
    _check(_load().qo_threshold(_ptr(s), ctypes.c_int64(M), ctypes.c_int64(N), _ptr(T), _ptr(f),
                                _ptr(bits)), "threshold")
    return bits


def bn_sign_direct(s, gamma: float, beta: float, mu: float, sigma: float) -> np.ndarray:
    s = _c(s, np.int32)
    bits = np.empty(s.shape, np.uint8)
    rc = _load().qo_bn_sign_direct(_ptr(s), ctypes.c_int64(s.size), ctypes.c_double(gamma),
                                   ctypes.c_double(beta), ctypes.c_double(mu), ctypes.c_double(sigma),
                                   _ptr(bits))
    _check(rc, "bn_sign_direct")
    return bits


def conv2d(X, Wt, stride: int = 1, pad: int = 1, pad_value: int = 1) -> np.ndarray:
    """+-1 cross-correlation, X [B,C,H,W], Wt [Cout,C,KH,KW] int32 -> [B,Cout,Ho,Wo]."""
    X = _c(X, np.int32)
    Wt = _c(Wt, np.int32)
    B, C, H, W = X.shape
    Cout, C2, KH, KW = Wt.shape
    assert C == C2
    Ho = (H + 2 * pad - KH) // stride + 1
    Wo = (W + 2 * pad - KW) // stride + 1
    out = np.empty((B, Cout, Ho, Wo), np.int32)
    rc = _load().qo_conv2d(_ptr(X), _ptr(Wt), B, C, H, W, Cout, KH, KW, stride, pad, pad_value, _ptr(out))
    _check(rc, "conv2d")
    return out


def ap2_exponent(x) -> np.ndarray:
    """round(log2|x|) of AP2 (Algorithm 2's caption); INT32_MIN for 0, INT32_MAX for inf / NaN."""
    x = _c(x, np.float32)
    e = np.empty(x.shape, np.int32)
    _check(_load().qo_ap2_exponent(_ptr(x), ctypes.c_int64(x.size), _ptr(e)), "ap2_exponent")
    return e


def log_quant(x, emin: int, emax: int) -> np.ndarray:
    """Eq. 10 with magnitudes clipped to [2^emin, 2^emax], as integers sign * 2^(e - emin)."""
    x = _c(x, np.float32)
    v = np.empty(x.shape, np.int32)
    _check(_load().qo_log_quant(_ptr(x), ctypes.c_int64(x.size), ctypes.c_int(emin), ctypes.c_int(emax), _ptr(v)),
           "log_quant")
    return v


def log_gemm(x, w, emin: int, emax: int) -> np.ndarray:
    """The backward products of Algorithm 1 with logarithmically quantised gradients (Eq. 10; Sec. 4.4 quantises
    them to 6 bits: a sign and up to 31 exponents): out[m,n] = sum_k LogQuant(x)[m,k] * w[k,n], exact, as int64 in
    units of 2^emin.  x: float [M,K]; w: integers [K,N] (the +-1 weights, or +-1 activations for the weight
    gradient).  The definition written out: quantise, then an integer matrix product (a library matmul on int64)."""
    if emax - emin > 30:
        raise ValueError("log_gemm: at most 31 exponents")
    v = log_quant(x, emin, emax).astype(np.int64)
    return v @ np.ascontiguousarray(w).astype(np.int64)


def maxpool2x2(x) -> np.ndarray:
    """2 x 2 / stride 2 max-pooling of an int32 [B,C,H,W] tensor (Table 7); odd tails dropped."""
    x = _c(x, np.int32)
    B, C, H, W = x.shape
    out = np.empty((B, C, H // 2, W // 2), np.int32)
    _check(_load().qo_maxpool2x2(_ptr(x), B, C, H, W, _ptr(out)), "maxpool2x2")
    return out


def convnet_forward(x, layers) -> np.ndarray:
    """The ConvNet of Table 7 at inference, in the table's order: convolution, (2 x 2 max-pooling,)
    batch norm folded to a threshold, binarisation; then the fully connected layers of Algorithm 4.

    x: integer codes [B,C,H,W] (8-bit pixels).  layers: dicts with
      kind 'conv': W +-1 int32 [Cout,C,k,k], pad, pad_value (what a tap outside the image reads:
                   0 for the pixel codes of the first layer, +1 for +-1 activations), pool (bool)
      kind 'fc'  : W +-1 int32 [K,N]; the first one reads the last feature map flattened in
                   (h, w, c) order
      T, flip    : folded thresholds of the layer; T None on the last layer (integer scores).
    Returns the last layer's int32 result."""
    a = _c(x, np.int32)
    for i, ly in enumerate(layers):
        if ly["kind"] == "conv":
            s = conv2d(a, ly["W"], 1, ly["pad"], ly["pad_value"])
            if ly.get("pool"):
                s = maxpool2x2(s)
            if ly.get("T") is None:
                return s
            Bq, Co, Ho, Wo = s.shape
            rows = s.transpose(0, 2, 3, 1).reshape(-1, Co)
            bits = threshold(rows, ly["T"], ly.get("flip"))
            a = np.where(bits.reshape(Bq, Ho, Wo, Co) != 0, 1, -1).astype(np.int32).transpose(0, 3, 1, 2)
        else:
            if a.ndim == 4:
                a = a.transpose(0, 2, 3, 1).reshape(a.shape[0], -1)
            s = int_gemm(a, ly["W"])
            if ly.get("T") is None:
                return s
            a = np.where(threshold(s, ly["T"], ly.get("flip")) != 0, 1, -1).astype(np.int32)
    return a


def mlp_forward(x, Ws: Sequence[np.ndarray], Ts: Sequence[np.ndarray],
                flips: Optional[Sequence[Optional[np.ndarray]]] = None) -> np.ndarray:
    """Algorithm 4: x int codes [M,K0]; Ws[l] +-1 int32 [K_l, K_{l+1}]; Ts[l] for l < L-1."""
    x = _c(x, np.int32)
    M = x.shape[0]
    L = len(Ws)
    Ws = [_c(w, np.int32) for w in Ws]
    Ts = [_c(t, np.int32) for t in Ts]
    assert len(Ts) == L - 1
    dims = np.array([x.shape[1]] + [w.shape[1] for w in Ws], np.int64)
    for l in range(L):
        assert Ws[l].shape[0] == dims[l]
    wp = (ctypes.c_void_p * L)(*[w.ctypes.data for w in Ws])
    tp = (ctypes.c_void_p * max(L - 1, 1))(*[t.ctypes.data for t in Ts])
    fl = None
    keep = []
    if flips is not None:
        arr = []
        for f in flips:
            if f is None:
                arr.append(None)
            else:
                fa = _c(f, np.uint8)
                keep.append(fa)
                arr.append(fa.ctypes.data)
        fl = (ctypes.c_void_p * max(L - 1, 1))(*arr)
    scores = np.empty((M, int(dims[-1])), np.int32)
    rc = _load().qo_mlp_forward(_ptr(x), ctypes.c_int64(M), ctypes.c_int(L), _ptr(dims), wp, tp, fl,
                                _ptr(scores))
    _check(rc, "mlp_forward")
    return scores


def rescale(p, alpha: float, row_off=None, col_off=None, delta: float = 0.0) -> np.ndarray:
    p = _c(p, np.int32)
    M, N = p.shape
    r = None if row_off is None else _c(row_off, np.float64)
    c = None if col_off is None else _c(col_off, np.float64)
    y = np.empty((M, N), np.float64)
    _check(_load().qo_rescale(_ptr(p), ctypes.c_int64(M), ctypes.c_int64(N), ctypes.c_double(alpha),
                              _ptr(r), _ptr(c), ctypes.c_double(delta), _ptr(y)), "rescale")
    return y
