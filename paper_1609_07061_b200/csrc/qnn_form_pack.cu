// Quantisers that write a tensor-core operand form directly from real tensors
// (Eq. 1 sign, Eq. 9 uniform k-bit): one pass over the fp32 data instead of
// "pack to bit-planes, then rewrite the planes one value per element".  The
// values and the layouts are exactly those qnn_tc_prepack produces from packed
// planes; pad elements up to the next multiple of 32 are written as 0.
// HBM-bound streaming kernels: 128-bit coalesced loads, a chunk's loads all in
// flight before the first conversion.
#include "qnn_internal.cuh"

namespace qnn {
namespace {

// value of one element: Eq. 1 gives +-1; Eq. 9 gives the code q (QNN_MODE_U01) or 2q - (2^bits - 1) (QNN_MODE_PM1)
struct SignValue {
    __device__ __forceinline__ int operator()(float v) const { return v >= 0.0f ? 1 : -1; }
};
struct KbitValue {
    float lo, hi, inv_step;
    int qmax, pm1;
    __device__ __forceinline__ int operator()(float t) const
    {
        // clip, subtract, multiply, round-half-even: separately rounded fp32 steps (NaN -> lo)
        t = fminf(fmaxf(t, lo), hi);
        const float d = __fsub_rn(t, lo);
        const float u = __fmul_rn(d, inv_step);
        int q = __float2int_rn(u);
        q = q < 0 ? 0 : (q > qmax ? qmax : q);
        return pm1 ? 2 * q - qmax : q;
    }
};

// e2m1 code of an integer in {0, +-1, +-2, +-3}: sign in bit 3; magnitudes 1 -> 0b010, 2 -> 0b100, 3 -> 0b101
__device__ __forceinline__ uint32_t e2m1_of(int v)
{
    const int m = v < 0 ? -v : v;
    return (uint32_t)(2 * m - (m == 3)) | (v < 0 ? 8u : 0u);
}

// four consecutive elements as form bytes: e2m1 -> 16 bits (element 0 in the lowest nibble), int8 -> 32 bits
template <int FORM>
__device__ __forceinline__ uint32_t encode4(int a, int b, int c, int d)
{
    if (FORM == QNN_FORM_FP4) return e2m1_of(a) | (e2m1_of(b) << 4) | (e2m1_of(c) << 8) | (e2m1_of(d) << 12);
    return ((uint32_t)a & 0xffu) | (((uint32_t)b & 0xffu) << 8) | (((uint32_t)c & 0xffu) << 16) | (((uint32_t)d & 0xffu) << 24);
}

// Row-major source [rows, K] -> form rows [rows, ld_bytes].  A warp owns a (row, chunk) pair, a chunk is 128 * UNROLL
// elements; lane l loads the 16-byte vectors at k0 + u*128 + 4*l and stores their 2 (e2m1) or 4 (int8) form bytes,
// so that a warp's stores of one u are 64 or 128 contiguous bytes.  Kz = K rounded up to 32: elements in [K, Kz) are 0.
template <class Value, int FORM, int UNROLL, bool VEC>
__global__ void __launch_bounds__(256, 4) row_form_kernel(const float *__restrict__ x, int64_t ldx, Value value, int64_t rows,
                                                          int64_t K, int64_t Kz, uint8_t *__restrict__ out, int64_t ld_bytes,
                                                          int64_t chunks_per_row)
{
    griddep_launch_dependents();
    griddep_wait();
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t total = rows * chunks_per_row;
    constexpr int CHUNK = 128 * UNROLL;
    for (int64_t item = warp0; item < total; item += nwarps) {
        const int64_t r = item / chunks_per_row;
        const int64_t k0 = (item - r * chunks_per_row) * CHUNK;
        const float *src = x + r * ldx;
        uint8_t *dst = out + r * ld_bytes;
        if (VEC && k0 + CHUNK <= K) {
            float4 raw[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) raw[u] = __ldcs(reinterpret_cast<const float4 *>(src + k0 + u * 128 + lane * 4));
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int64_t k = k0 + u * 128 + lane * 4;
                const uint32_t e = encode4<FORM>(value(raw[u].x), value(raw[u].y), value(raw[u].z), value(raw[u].w));
                if (FORM == QNN_FORM_FP4) *reinterpret_cast<uint16_t *>(dst + (k >> 1)) = (uint16_t)e;
                else *reinterpret_cast<uint32_t *>(dst + k) = e;
            }
        } else {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int64_t k = k0 + u * 128 + lane * 4;
                if (k >= Kz) continue;
                int v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) v[j] = (k + j < K) ? value(src[k + j]) : 0;
                const uint32_t e = encode4<FORM>(v[0], v[1], v[2], v[3]);
                if (FORM == QNN_FORM_FP4) *reinterpret_cast<uint16_t *>(dst + (k >> 1)) = (uint16_t)e;
                else *reinterpret_cast<uint32_t *>(dst + k) = e;
            }
        }
    }
}

template <class Value, int FORM>
int launch_row_form(const float *x, int64_t ldx, const Value &value, int64_t rows, int64_t K, uint8_t *out, int64_t ld_bytes,
                    cudaStream_t st, const char *what)
{
    constexpr int UNROLL = 8;
    const int64_t Kz = (int64_t)round_up((size_t)K, 32);
    const int64_t chunks = ceil_div(K, 128 * UNROLL);
    const int64_t blocks_needed = ceil_div(rows * chunks, 8);
    const int64_t cap = (int64_t)sm_count() * 4;
    const int blocks = (int)(blocks_needed < cap ? blocks_needed : cap);
    const bool vec = (ldx % 4 == 0) && aligned(x, 16);
    if (vec)
        QNN_CUDA(launch_pdl(row_form_kernel<Value, FORM, UNROLL, true>, dim3(blocks), dim3(256), 0, st, x, ldx, value, rows, K, Kz, out,
                            ld_bytes, chunks));
    else
        QNN_CUDA(launch_pdl(row_form_kernel<Value, FORM, UNROLL, false>, dim3(blocks), dim3(256), 0, st, x, ldx, value, rows, K, Kz, out,
                            ld_bytes, chunks));
    return check_launch(what);
}

// Transposed source [batch][K, N] (row-major, K strided) -> form rows [batch][N, ld_bytes] along K.  A thread owns 4
// neighbouring n and 32 consecutive k: every load is a 16-byte vector along n, coalesced across the warp, sixteen in
// flight per thread; it ends up holding the 16 (e2m1) or 32 (int8) form bytes of each of its four rows.
template <class Value, int FORM, bool VEC>
__global__ void __launch_bounds__(128) trans_form_kernel(const float *__restrict__ w, int64_t K, int64_t N, int64_t ldw,
                                                         int64_t batch_stride_in, Value value, uint8_t *__restrict__ out,
                                                         int64_t ld_bytes, int64_t batch_stride_out)
{
    griddep_launch_dependents();
    griddep_wait();
    const int64_t n0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    const int64_t kw = blockIdx.y;
    const int64_t bz = blockIdx.z;
    if (n0 >= N) return;
    const float *src = w + bz * batch_stride_in;
    constexpr int WORDS = FORM == QNN_FORM_FP4 ? 4 : 8;          // 32-bit words of form per 32 elements
    constexpr int PER = 32 / WORDS;                              // elements per word: 8 nibbles or 4 bytes
    constexpr int SH = FORM == QNN_FORM_FP4 ? 4 : 8;
    uint32_t word[4][WORDS];
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < WORDS; ++i) word[c][i] = 0;
    const int64_t kbase = kw * 32;
    auto put = [&](int c, int j, float f) {
        const int v = value(f);
        const uint32_t e = FORM == QNN_FORM_FP4 ? e2m1_of(v) : ((uint32_t)v & 0xffu);
        word[c][j / PER] |= e << (SH * (j % PER));
    };
    if (VEC && n0 + 4 <= N && kbase + 32 <= K) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float4 t[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) t[j] = __ldcs(reinterpret_cast<const float4 *>(src + (kbase + h * 16 + j) * ldw + n0));
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                put(0, h * 16 + j, t[j].x); put(1, h * 16 + j, t[j].y); put(2, h * 16 + j, t[j].z); put(3, h * 16 + j, t[j].w);
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const int64_t k = kbase + j;
            if (k < K) {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (n0 + c < N) put(c, j, src[k * ldw + n0 + c]);
            }
        }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        if (n0 + c < N) {
            uint4 *dst = reinterpret_cast<uint4 *>(out + bz * batch_stride_out + (n0 + c) * ld_bytes + kw * (4 * WORDS));
            dst[0] = make_uint4(word[c][0], word[c][1], word[c][2], word[c][3]);
            if (FORM == QNN_FORM_I8) dst[1] = make_uint4(word[c][WORDS - 4], word[c][WORDS - 3], word[c][WORDS - 2], word[c][WORDS - 1]);
        }
    }
}

template <class Value, int FORM>
int launch_trans_form(const float *w, int64_t K, int64_t N, int64_t ldw, int64_t batch, int64_t bs_in, const Value &value,
                      uint8_t *out, int64_t ld_bytes, int64_t bs_out, cudaStream_t st, const char *what)
{
    const int64_t kwords = ceil_div(K, 32);
    QNN_REQUIRE(kwords <= 65535 && batch <= 65535, QNN_ERR_UNSUPPORTED, "%s: K/32 or batch exceeds 65535", what);
    dim3 grid((unsigned)ceil_div(N, 128 * 4), (unsigned)kwords, (unsigned)batch);
    const bool vec = (ldw % 4 == 0) && (bs_in % 4 == 0) && aligned(w, 16);
    if (vec)
        QNN_CUDA(launch_pdl(trans_form_kernel<Value, FORM, true>, grid, dim3(128), 0, st, w, K, N, ldw, bs_in, value, out, ld_bytes, bs_out));
    else
        QNN_CUDA(launch_pdl(trans_form_kernel<Value, FORM, false>, grid, dim3(128), 0, st, w, K, N, ldw, bs_in, value, out, ld_bytes, bs_out));
    return check_launch(what);
}

int check_form_out(const char *what, int form, int planes, int mode, int64_t K, const void *out, int64_t ld_bytes)
{
    QNN_REQUIRE(form == QNN_FORM_I8 || form == QNN_FORM_FP4, QNN_ERR_INVALID_ARG, "%s: unknown form %d", what, form);
    QNN_REQUIRE(mode == QNN_MODE_U01 || mode == QNN_MODE_PM1, QNN_ERR_INVALID_ARG, "%s: unknown value mode %d", what, mode);
    QNN_REQUIRE(tc_form_holds(form, planes, mode), QNN_ERR_UNSUPPORTED, "%s: %d-bit values do not fit form %d", what, planes, form);
    QNN_REQUIRE(aligned(out, 16) && ld_bytes % 16 == 0 && ld_bytes >= tc_row_bytes(ceil_div(K, 32), form), QNN_ERR_ALIGNMENT,
                "%s: out needs a 16-byte aligned base and a row stride that is a multiple of 16 covering K", what);
    return QNN_OK;
}

template <class Value>
int dispatch_row(int form, const float *x, int64_t ldx, const Value &v, int64_t rows, int64_t K, void *out, int64_t ld_bytes,
                 cudaStream_t st, const char *what)
{
    if (form == QNN_FORM_FP4) return launch_row_form<Value, QNN_FORM_FP4>(x, ldx, v, rows, K, static_cast<uint8_t *>(out), ld_bytes, st, what);
    return launch_row_form<Value, QNN_FORM_I8>(x, ldx, v, rows, K, static_cast<uint8_t *>(out), ld_bytes, st, what);
}
template <class Value>
int dispatch_trans(int form, const float *w, int64_t K, int64_t N, int64_t ldw, int64_t batch, int64_t bs_in, const Value &v, void *out,
                   int64_t ld_bytes, int64_t bs_out, cudaStream_t st, const char *what)
{
    if (form == QNN_FORM_FP4)
        return launch_trans_form<Value, QNN_FORM_FP4>(w, K, N, ldw, batch, bs_in, v, static_cast<uint8_t *>(out), ld_bytes, bs_out, st, what);
    return launch_trans_form<Value, QNN_FORM_I8>(w, K, N, ldw, batch, bs_in, v, static_cast<uint8_t *>(out), ld_bytes, bs_out, st, what);
}

int make_kbit(const char *what, int bits, float lo, float hi, int mode, KbitValue *v)
{
    QNN_REQUIRE(bits >= 1 && bits <= 8, QNN_ERR_INVALID_ARG, "%s: bits must be in 1..8", what);
    QNN_REQUIRE(hi > lo, QNN_ERR_INVALID_ARG, "%s: need hi > lo", what);
    v->lo = lo; v->hi = hi; v->qmax = (1 << bits) - 1; v->pm1 = mode == QNN_MODE_PM1;
    v->inv_step = (float)((1 << bits) - 1) / (hi - lo);
    return QNN_OK;
}

}  // namespace
}  // namespace qnn

using namespace qnn;

extern "C" {

int qnn_quantize_form_sign(const float *x, int64_t rows, int64_t K, int64_t ldx, int form, void *out, int64_t ld_bytes, void *stream)
{
    const char *what = "qnn_quantize_form_sign";
    QNN_REQUIRE(rows >= 0 && K >= 0, QNN_ERR_INVALID_ARG, "%s: negative size", what);
    if (rows == 0 || K == 0) return QNN_OK;
    QNN_REQUIRE(x && out && ldx >= K, QNN_ERR_INVALID_ARG, "%s: NULL pointer or ldx below K", what);
    if (int rc = check_form_out(what, form, 1, QNN_MODE_PM1, K, out, ld_bytes)) return rc;
    return dispatch_row(form, x, ldx, SignValue{}, rows, K, out, ld_bytes, as_stream(stream), what);
}

int qnn_quantize_form_sign_t(const float *w, int64_t K, int64_t N, int64_t ldw, int form, void *out, int64_t ld_bytes, void *stream)
{
    const char *what = "qnn_quantize_form_sign_t";
    QNN_REQUIRE(K >= 0 && N >= 0, QNN_ERR_INVALID_ARG, "%s: negative size", what);
    if (K == 0 || N == 0) return QNN_OK;
    QNN_REQUIRE(w && out && ldw >= N, QNN_ERR_INVALID_ARG, "%s: NULL pointer or ldw below N", what);
    if (int rc = check_form_out(what, form, 1, QNN_MODE_PM1, K, out, ld_bytes)) return rc;
    return dispatch_trans(form, w, K, N, ldw, 1, 0, SignValue{}, out, ld_bytes, 0, as_stream(stream), what);
}

int qnn_quantize_form_sign_nchw(const float *x, int B, int C, int H, int W, int form, void *out, int64_t ld_bytes, void *stream)
{
    const char *what = "qnn_quantize_form_sign_nchw";
    QNN_REQUIRE(B >= 0 && C >= 0 && H >= 0 && W >= 0, QNN_ERR_INVALID_ARG, "%s: negative size", what);
    if (B == 0 || C == 0 || H == 0 || W == 0) return QNN_OK;
    QNN_REQUIRE(x && out, QNN_ERR_INVALID_ARG, "%s: NULL pointer", what);
    if (int rc = check_form_out(what, form, 1, QNN_MODE_PM1, C, out, ld_bytes)) return rc;
    // per image: a [C, H*W] matrix turned into H*W rows along C
    const int64_t hw = (int64_t)H * W;
    return dispatch_trans(form, x, C, hw, hw, B, (int64_t)C * hw, SignValue{}, out, ld_bytes, hw * ld_bytes, as_stream(stream), what);
}

int qnn_quantize_form_kbit(const float *x, int64_t rows, int64_t K, int64_t ldx, int bits, float lo, float hi, int mode, int form,
                           void *out, int64_t ld_bytes, void *stream)
{
    const char *what = "qnn_quantize_form_kbit";
    QNN_REQUIRE(rows >= 0 && K >= 0, QNN_ERR_INVALID_ARG, "%s: negative size", what);
    KbitValue v;
    if (int rc = make_kbit(what, bits, lo, hi, mode, &v)) return rc;
    if (rows == 0 || K == 0) return QNN_OK;
    QNN_REQUIRE(x && out && ldx >= K, QNN_ERR_INVALID_ARG, "%s: NULL pointer or ldx below K", what);
    if (int rc = check_form_out(what, form, bits, mode, K, out, ld_bytes)) return rc;
    return dispatch_row(form, x, ldx, v, rows, K, out, ld_bytes, as_stream(stream), what);
}

int qnn_quantize_form_kbit_t(const float *w, int64_t K, int64_t N, int64_t ldw, int bits, float lo, float hi, int mode, int form,
                             void *out, int64_t ld_bytes, void *stream)
{
    const char *what = "qnn_quantize_form_kbit_t";
    QNN_REQUIRE(K >= 0 && N >= 0, QNN_ERR_INVALID_ARG, "%s: negative size", what);
    KbitValue v;
    if (int rc = make_kbit(what, bits, lo, hi, mode, &v)) return rc;
    if (K == 0 || N == 0) return QNN_OK;
    QNN_REQUIRE(w && out && ldw >= N, QNN_ERR_INVALID_ARG, "%s: NULL pointer or ldw below N", what);
    if (int rc = check_form_out(what, form, bits, mode, K, out, ld_bytes)) return rc;
    return dispatch_trans(form, w, K, N, ldw, 1, 0, v, out, ld_bytes, 0, as_stream(stream), what);
}

}  // extern "C"
