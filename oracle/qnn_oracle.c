/*
 * qnn_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, scalar CPU statement of what the quantised-network forward
 * path computes, written from the paper's definitions.  It works on UNPACKED
 * values (one int per +-1 value or integer code, one byte per output bit),
 * uses no bit tricks, and shares no code with the CUDA library.  Only the
 * tests, the smoke check and the benchmark's cpu baseline may call it.
 *
 * Integer results are exact; every sum is accumulated in int64 and checked
 * to fit int32 before it is stored.  Floating-point decisions (sign, the
 * k-bit quantiser) are taken in fp32 with one IEEE operation per step
 * (compile with -ffp-contract=off).
 *
 * Parallelism: an OpenMP "parallel for" over independent output rows only.
 *
 * Every function returns 0 on success, 1 on int32 overflow of a result,
 * 2 on an invalid argument.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int qo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Eq. 1: deterministic binarisation.  x >= 0 gives +1, everything else
 * (negative numbers and NaN, for which the comparison is false) gives -1.
 * Both +0.0 and -0.0 compare >= 0 and give +1. */
static int sgn(float x) { return (x >= 0.0f) ? 1 : -1; }

int qo_sign(const float *x, int64_t n, int32_t *out)
{
    if (n < 0) return 2;
    for (int64_t i = 0; i < n; ++i) out[i] = sgn(x[i]);
    return 0;
}

/* Eq. 9 read as a uniform quantiser with 2^bits levels on [lo, hi]:
 * clip, then round (x - lo) / step to the nearest integer code, ties to even.
 * inv_step = (2^bits - 1) / (hi - lo) is computed once by the caller in fp32
 * and handed to both implementations.  NaN clips to lo (code 0). */
int qo_linear_quant_codes(const float *x, int64_t n, int bits, float lo, float hi, float inv_step,
                          int32_t *q)
{
    if (n < 0 || bits < 1 || bits > 8 || !(hi > lo)) return 2;
    const int32_t qmax = (1 << bits) - 1;
    for (int64_t i = 0; i < n; ++i) {
        float t = x[i];
        if (!(t >= lo)) t = lo;
        if (t > hi) t = hi;
        float d = t - lo;
        float u = d * inv_step;
        int32_t c = (int32_t)nearbyintf(u); /* default rounding mode: half to even */
        if (c < 0) c = 0;
        if (c > qmax) c = qmax;
        q[i] = c;
    }
    return 0;
}

/* Signed-symmetric reading of a k-bit code: v = 2q - (2^bits - 1), an odd
 * integer in [-(2^bits-1), 2^bits-1]; equals sum_i 2^i * s_i with s_i = +-1
 * given by bit i of q. */
int qo_codes_to_symmetric(const int32_t *q, int64_t n, int bits, int32_t *v)
{
    if (n < 0 || bits < 1 || bits > 8) return 2;
    const int32_t L = (1 << bits) - 1;
    for (int64_t i = 0; i < n; ++i) v[i] = 2 * q[i] - L;
    return 0;
}

/* Eq. 8 / Algorithm 4, first layer: bit-plane n (1-based in the paper) of an
 * integer code is bit n-1 of its binary expansion; plane index i = n-1 here. */
int qo_bit_plane(const int32_t *q, int64_t n, int i, uint8_t *plane)
{
    if (n < 0 || i < 0 || i > 30) return 2;
    for (int64_t j = 0; j < n; ++j) plane[j] = (uint8_t)((q[j] / (1 << i)) % 2);
    return 0;
}

/* Plain integer matrix product  out[m,n] = sum_k A[m,k] * B[k,n].
 * A is [M,K] row-major, B is [K,N] row-major (the paper's a.W orientation).
 * The k loop is outermost within a row so B is read along its rows; the sum
 * itself is the textbook one. */
int qo_int_gemm(const int32_t *A, const int32_t *B, int64_t M, int64_t N, int64_t K, int32_t *out)
{
    if (M < 0 || N < 0 || K < 0) return 2;
    int overflow = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(| : overflow)
    for (int64_t m = 0; m < M; ++m) {
        int64_t *acc = (int64_t *)calloc((size_t)(N > 0 ? N : 1), sizeof(int64_t));
        for (int64_t k = 0; k < K; ++k) {
            const int64_t a = A[m * K + k];
            const int32_t *brow = B + k * N;
            for (int64_t n = 0; n < N; ++n) acc[n] += a * (int64_t)brow[n];
        }
        for (int64_t n = 0; n < N; ++n) {
            if (acc[n] > INT32_MAX || acc[n] < INT32_MIN) overflow |= 1;
            out[m * N + n] = (int32_t)acc[n];
        }
        free(acc);
    }
    return overflow;
}

/* Algorithm 4 hidden layer, "XnorDotProduct" of two real tensors after Eq. 1:
 * Y[m,n] = sum_k sign(X[m,k]) * sign(W[k,n]). */
int qo_xnor_gemm(const float *X, const float *W, int64_t M, int64_t N, int64_t K, int32_t *Y)
{
    if (M < 0 || N < 0 || K < 0) return 2;
    int32_t *xs = (int32_t *)malloc(sizeof(int32_t) * (size_t)(M * K + 1));
    int32_t *ws = (int32_t *)malloc(sizeof(int32_t) * (size_t)(K * N + 1));
    qo_sign(X, M * K, xs);
    qo_sign(W, K * N, ws);
    int rc = qo_int_gemm(xs, ws, M, N, K, Y);
    free(xs);
    free(ws);
    return rc;
}

/* Eq. 8 evaluated literally, plane by plane:
 * out[m,n] = sum_{i<ka} 2^i * ( plane_i(QA)[m,:] . B[:,n] ),
 * with plane values 0/1.  Exists to check qo_int_gemm against Eq. 8; B holds
 * integer values (e.g. +-1 weights). */
int qo_planewise_gemm(const int32_t *QA, int ka, const int32_t *B, int64_t M, int64_t N, int64_t K,
                      int32_t *out)
{
    if (M < 0 || N < 0 || K < 0 || ka < 1 || ka > 8) return 2;
    int overflow = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(| : overflow)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            int64_t s = 0;
            for (int i = 0; i < ka; ++i) {
                int64_t dot = 0;
                for (int64_t k = 0; k < K; ++k) {
                    int64_t bit = (QA[m * K + k] / (1 << i)) % 2;
                    dot += bit * (int64_t)B[k * N + n];
                }
                s += (int64_t)(1 << i) * dot;
            }
            if (s > INT32_MAX || s < INT32_MIN) overflow |= 1;
            out[m * N + n] = (int32_t)s;
        }
    }
    return overflow;
}

/* AP2 (caption of Algorithm 2): AP2(x) = sign(x) * 2^round(log2|x|), returned as the exponent e = round(log2|x|).
 * |x| = m * 2^f with m in [1, 2) (frexpf gives m/2 and f+1): log2|x| = f + log2 m, and log2 m >= 1/2 exactly when
 * m >= sqrt(2).  sqrt(2) is not a float, so no input sits on the tie: m rounds up when it is above the largest
 * float below sqrt(2).  x = 0 has no logarithm: e = INT32_MIN (it clips to the smallest level in Eq. 10);
 * infinities and NaN give INT32_MAX (they clip to the largest). */
static int32_t ap2_exponent(float x)
{
    float ax = fabsf(x);
    if (!(ax == ax) || isinf(ax)) return INT32_MAX;
    if (ax == 0.0f) return INT32_MIN;
    int f;
    float half_m = frexpf(ax, &f);          /* ax = half_m * 2^f, half_m in [0.5, 1) */
    float m = half_m * 2.0f;                /* exact */
    int32_t e = f - 1;
    const float below_sqrt2 = 1.41421353816986083984375f;   /* largest float < sqrt(2) */
    if (m > below_sqrt2) e += 1;
    return e;
}

int qo_ap2_exponent(const float *x, int64_t n, int32_t *e)
{
    if (n < 0) return 2;
    for (int64_t i = 0; i < n; ++i) e[i] = ap2_exponent(x[i]);
    return 0;
}

/* Eq. 10: LogQuant(x) = Clip(AP2(x), minV, maxV) with minV = 2^emin, maxV = 2^emax as bounds on the magnitude.
 * The result is returned as the integer v = sign * 2^(e - emin), e = clamp(round(log2|x|), emin, emax), i.e. the
 * quantised value in units of minV: |v| in {1, 2, 4, ..., 2^(emax-emin)}; sign as in Eq. 1 (x >= 0 gives +1). */
int qo_log_quant(const float *x, int64_t n, int emin, int emax, int32_t *v)
{
    if (n < 0 || emax < emin || emax - emin > 30) return 2;
    for (int64_t i = 0; i < n; ++i) {
        int32_t e = ap2_exponent(x[i]);
        if (e < emin) e = emin;
        if (e > emax) e = emax;
        v[i] = sgn(x[i]) * (int32_t)(1 << (e - emin));
    }
    return 0;
}

/* Algorithm 4: a^b = Sign(BatchNorm(a, theta)) with the batch-norm folded to a
 * per-channel integer comparison: bit = (s >= T[n]) xor flip[n].  Output is
 * one byte (0/1) per element, not packed.  flip may be NULL (all zero). */
int qo_threshold(const int32_t *s, int64_t M, int64_t N, const int32_t *T, const uint8_t *flip,
                 uint8_t *bits)
{
    if (M < 0 || N < 0) return 2;
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            int ge = s[m * N + n] >= T[n];
            int f = flip ? (flip[n] != 0) : 0;
            bits[m * N + n] = (uint8_t)(ge != f);
        }
    return 0;
}

/* Inference-time batch norm followed by Eq. 1, evaluated directly in double:
 * y = gamma * (s - mu) / sigma + beta ; bit = (y >= 0).  Used to check the
 * threshold fold. */
int qo_bn_sign_direct(const int32_t *s, int64_t n, double gamma, double beta, double mu,
                      double sigma, uint8_t *bits)
{
    if (n < 0 || !(sigma > 0.0)) return 2;
    for (int64_t i = 0; i < n; ++i) {
        double y = gamma * (((double)s[i] - mu) / sigma) + beta;
        bits[i] = (uint8_t)(y >= 0.0);
    }
    return 0;
}

/* Binary 2-D convolution as the same +-1 multiply-accumulate per filter tap
 * (cross-correlation, zero-based tap offsets kh - pad, kw - pad):
 * out[b,co,y,x] = sum_{ci,kh,kw} xs[b,ci,y*stride+kh-pad,x*stride+kw-pad] * ws[co,ci,kh,kw]
 * where xs, ws are +-1 values and a tap outside the image reads pad_value.
 * X is [B,C,H,W], Wt is [Cout,C,KH,KW], out is [B,Cout,Ho,Wo], all row-major. */
int qo_conv2d(const int32_t *X, const int32_t *Wt, int B, int C, int H, int W, int Cout, int KH,
              int KW, int stride, int pad, int pad_value, int32_t *out)
{
    if (B < 0 || C < 0 || H < 1 || W < 1 || Cout < 0 || KH < 1 || KW < 1 || stride < 1 || pad < 0)
        return 2;
    const int Ho = (H + 2 * pad - KH) / stride + 1;
    const int Wo = (W + 2 * pad - KW) / stride + 1;
    int overflow = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1) reduction(| : overflow)
    for (int b = 0; b < B; ++b)
        for (int co = 0; co < Cout; ++co)
            for (int y = 0; y < Ho; ++y)
                for (int x = 0; x < Wo; ++x) {
                    int64_t s = 0;
                    for (int ci = 0; ci < C; ++ci)
                        for (int kh = 0; kh < KH; ++kh)
                            for (int kw = 0; kw < KW; ++kw) {
                                int yy = y * stride + kh - pad;
                                int xx = x * stride + kw - pad;
                                int64_t xv = pad_value;
                                if (yy >= 0 && yy < H && xx >= 0 && xx < W)
                                    xv = X[(((int64_t)b * C + ci) * H + yy) * W + xx];
                                s += xv * Wt[(((int64_t)co * C + ci) * KH + kh) * KW + kw];
                            }
                    if (s > INT32_MAX || s < INT32_MIN) overflow |= 1;
                    out[(((int64_t)b * Cout + co) * Ho + y) * Wo + x] = (int32_t)s;
                }
    return overflow;
}

/* 2 x 2 max-pooling with stride 2 of an int32 [B,C,H,W] tensor, the pooling that
 * Table 7 places between a convolution and its batch norm.  A trailing odd row
 * or column is dropped: out is [B,C,H/2,W/2] (integer division). */
int qo_maxpool2x2(const int32_t *x, int B, int C, int H, int W, int32_t *out)
{
    if (B < 0 || C < 0 || H < 0 || W < 0) return 2;
    const int Ho = H / 2, Wo = W / 2;
    for (int64_t bc = 0; bc < (int64_t)B * C; ++bc)
        for (int y = 0; y < Ho; ++y)
            for (int xo = 0; xo < Wo; ++xo) {
                const int32_t *p = x + (bc * H + 2 * y) * W + 2 * xo;
                int32_t m = p[0];
                if (p[1] > m) m = p[1];
                if (p[W] > m) m = p[W];
                if (p[W + 1] > m) m = p[W + 1];
                out[(bc * Ho + y) * Wo + xo] = m;
            }
    return 0;
}

/* Algorithm 4 in full for an MLP whose input is an unsigned integer code
 * (8-bit pixels in the paper):
 *   layer 1:      a_1 = x . W_1            (integer x, +-1 weights; Eq. 8)
 *   layers 1..L-1: a^b = threshold(a)      (+1 where bit = 1, -1 where bit = 0)
 *   layers 2..L:  a_k = a^b_{k-1} . W_k
 * The last layer's integer scores are returned; its affine batch norm is left
 * to the caller.  Ws[l] is the +-1 matrix [dims[l], dims[l+1]]; T[l], flip[l]
 * are the folded thresholds of layer l (l < L-1); flip[l] may be NULL. */
int qo_mlp_forward(const int32_t *x, int64_t M, int L, const int64_t *dims,
                   const int32_t *const *Ws, const int32_t *const *T, const uint8_t *const *flip,
                   int32_t *scores)
{
    if (L < 1 || M < 0) return 2;
    int64_t maxd = 0;
    for (int l = 0; l <= L; ++l)
        if (dims[l] > maxd) maxd = dims[l];
    int32_t *act = (int32_t *)malloc(sizeof(int32_t) * (size_t)(M * maxd + 1));
    int32_t *pre = (int32_t *)malloc(sizeof(int32_t) * (size_t)(M * maxd + 1));
    uint8_t *bit = (uint8_t *)malloc((size_t)(M * maxd + 1));
    memcpy(act, x, sizeof(int32_t) * (size_t)(M * dims[0]));
    int rc = 0;
    for (int l = 0; l < L; ++l) {
        int32_t *dst = (l == L - 1) ? scores : pre;
        rc |= qo_int_gemm(act, Ws[l], M, dims[l + 1], dims[l], dst);
        if (l < L - 1) {
            rc |= qo_threshold(pre, M, dims[l + 1], T[l], flip ? flip[l] : NULL, bit);
            for (int64_t i = 0; i < M * dims[l + 1]; ++i) act[i] = bit[i] ? 1 : -1;
        }
    }
    free(act);
    free(pre);
    free(bit);
    return rc;
}

/* Affine rescale of an integer result, in double:
 * y[m,n] = alpha * p[m,n] + row_off[m] + col_off[n] + delta  (offsets may be NULL). */
int qo_rescale(const int32_t *p, int64_t M, int64_t N, double alpha, const double *row_off,
               const double *col_off, double delta, double *y)
{
    if (M < 0 || N < 0) return 2;
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n)
            y[m * N + n] = alpha * (double)p[m * N + n] + (row_off ? row_off[m] : 0.0) +
                           (col_off ? col_off[n] : 0.0) + delta;
    return 0;
}
