// Logarithmic codes wider than an int8 value (Eq. 10 with up to 31 exponents: the 6-bit gradients of Sec. 4.4), for
// the backward products of Algorithm 1 -- gradient times +-1 weights, +-1 activations times gradient -- on the int8
// tensor-core form.
//
// A code sign * 2^(e - emin), e - emin in 0..30, does not fit an int8 value, but it has ONE set bit: the exponents are
// cut into groups of seven, group g holding sign * 2^((e - emin) - 7 g) where the exponent falls into it and 0
// elsewhere.  The G group matrices are stacked row-wise into one int8 operand of G * rows rows; ONE product with the
// +-1 matrix gives G blocks of int32 partial sums (each at most K * 64), and
//     out[m, n] = sum_g 2^(7 g) * P[g * rows + m, n]
// is the exact sum in int64.  The cost is G products' worth of int8 work -- the paper's cost model for wider codes (one
// pass of the binary kernel per bit, Sec. 3 and the end of Sec. 5) with seven bits per pass instead of one.
#include "qnn_internal.cuh"

namespace qnn {
namespace {

constexpr int LOG_GROUP = 7;                   // exponents per int8 group: 2^0 .. 2^6

// round(log2|x|) from the float's own fields, clipped to [emin, emax]; returned relative to emin, the sign (Eq. 1:
// x >= 0 is +1, NaN -1) in bit 31.  Zero and denormals clip to emin, infinities and NaN to emax.
__device__ __forceinline__ uint32_t log_code(float x, int emin, int emax)
{
    const uint32_t a = __float_as_uint(x) & 0x7fffffffu;
    int e;
    if (a >= 0x7f800000u) e = emax;
    else if (a < 0x00800000u) e = emin;
    else {
        e = (int)(a >> 23) - 127 + (int)((a & 0x7fffffu) > 0x3504f3u);     // mantissa above the largest float below sqrt(2)
        e = e < emin ? emin : (e > emax ? emax : e);
    }
    return (uint32_t)(e - emin) | (x >= 0.0f ? 0u : 0x80000000u);
}
__device__ __forceinline__ uint32_t group_byte(uint32_t code, int g)
{
    const int e = (int)(code & 0xffu) - LOG_GROUP * g;
    if (e < 0 || e >= LOG_GROUP) return 0u;
    const int v = 1 << e;
    return (uint32_t)((code >> 31) ? -v : v) & 0xffu;
}

// rows of x are rows of the operand: one thread per four consecutive elements of a row, all groups
__global__ void __launch_bounds__(256) log_groups_kernel(const float *__restrict__ x, int64_t rows, int64_t K, int64_t ldx, int emin,
                                                         int emax, int groups, uint8_t *__restrict__ out, int64_t ld_bytes, int64_t kq, bool vec)
{
    const int64_t total = rows * kq;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / kq, k = (i - r * kq) * 4;
        uint32_t c[4];
        if (vec && k + 4 <= K) {
            const float4 v = __ldcs(reinterpret_cast<const float4 *>(x + r * ldx + k));
            c[0] = log_code(v.x, emin, emax); c[1] = log_code(v.y, emin, emax); c[2] = log_code(v.z, emin, emax); c[3] = log_code(v.w, emin, emax);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) c[j] = k + j < K ? log_code(__ldcs(x + r * ldx + k + j), emin, emax) : 0xffu;   // 0xff: in no group
        }
        for (int g = 0; g < groups; ++g) {
            const uint32_t w = group_byte(c[0], g) | (group_byte(c[1], g) << 8) | (group_byte(c[2], g) << 16) | (group_byte(c[3], g) << 24);
            *reinterpret_cast<uint32_t *>(out + ((int64_t)g * rows + r) * ld_bytes + k) = w;
        }
    }
}

// columns of x [K, rows] are rows of the operand: 32 x 32 tiles through shared memory (reads along x's rows, writes
// along the operand's)
__global__ void __launch_bounds__(256) log_groups_t_kernel(const float *__restrict__ x, int64_t rows, int64_t K, int64_t ldx, int emin,
                                                           int emax, int groups, uint8_t *__restrict__ out, int64_t ld_bytes)
{
    __shared__ uint32_t tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t k0 = (int64_t)blockIdx.x * 32, n0 = (int64_t)blockIdx.y * 32;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t k = k0 + ty + 8 * i, n = n0 + tx;
        tile[ty + 8 * i][tx] = (k < K && n < rows) ? log_code(__ldcs(x + k * ldx + n), emin, emax) : 0xffu;
    }
    __syncthreads();
    // one thread per (operand row, four consecutive k) of the tile: a 4-byte store per group, eight threads to a 32-byte run
    const int nl = threadIdx.x >> 3, kq = threadIdx.x & 7;
    const int64_t n = n0 + nl;
    if (n >= rows) return;
    const uint32_t c0 = tile[4 * kq][nl], c1 = tile[4 * kq + 1][nl], c2 = tile[4 * kq + 2][nl], c3 = tile[4 * kq + 3][nl];
    for (int g = 0; g < groups; ++g)
        *reinterpret_cast<uint32_t *>(out + ((int64_t)g * rows + n) * ld_bytes + k0 + 4 * kq) =
            group_byte(c0, g) | (group_byte(c1, g) << 8) | (group_byte(c2, g) << 16) | (group_byte(c3, g) << 24);
}

// four consecutive columns per thread where the rows allow 16-byte accesses (the pass is a stream: 20 bytes in and 8 out
// per element)
template <bool VEC>
__global__ void __launch_bounds__(256) log_combine_kernel(const int32_t *__restrict__ p, int groups, int64_t M, int64_t N, int64_t ldp,
                                                          int64_t *__restrict__ out, int64_t ldo)
{
    const int64_t nq = VEC ? N / 4 : N;
    const int64_t total = M * nq;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t m = i / nq, n = (i - m * nq) * (VEC ? 4 : 1);
        if (VEC) {
            int64_t acc[4] = {0, 0, 0, 0};
            int4 v[5];
#pragma unroll
            for (int g = 0; g < 5; ++g)
                if (g < groups) v[g] = __ldcs(reinterpret_cast<const int4 *>(p + ((int64_t)g * M + m) * ldp + n));
#pragma unroll
            for (int g = 0; g < 5; ++g) {
                if (g < groups) {
                    acc[0] += (int64_t)v[g].x << (LOG_GROUP * g); acc[1] += (int64_t)v[g].y << (LOG_GROUP * g);
                    acc[2] += (int64_t)v[g].z << (LOG_GROUP * g); acc[3] += (int64_t)v[g].w << (LOG_GROUP * g);
                }
            }
            longlong2 *dst = reinterpret_cast<longlong2 *>(out + m * ldo + n);
            __stcs(dst, make_longlong2(acc[0], acc[1]));
            __stcs(dst + 1, make_longlong2(acc[2], acc[3]));
        } else {
            int64_t acc = 0;
            for (int g = 0; g < groups; ++g) acc += (int64_t)__ldcs(p + ((int64_t)g * M + m) * ldp + n) << (LOG_GROUP * g);
            out[m * ldo + n] = acc;
        }
    }
}

}  // namespace
}  // namespace qnn

using namespace qnn;

extern "C" {

int qnn_logquant_groups(int emin, int emax)
{
    if (emax < emin || emax - emin > 30) return 0;
    return (emax - emin) / LOG_GROUP + 1;
}

int qnn_logquant_pack_groups(const float *x, int64_t rows, int64_t K, int64_t ldx, int transposed, int emin, int emax, void *out,
                             int64_t ld_bytes, void *stream)
{
    const char *what = "qnn_logquant_pack_groups";
    QNN_REQUIRE(rows >= 0 && K >= 0, QNN_ERR_INVALID_ARG, "%s: negative size", what);
    QNN_REQUIRE(emax >= emin && emin >= -126 && emax <= 127, QNN_ERR_INVALID_ARG, "%s: need -126 <= emin <= emax <= 127", what);
    QNN_REQUIRE(emax - emin <= 30, QNN_ERR_UNSUPPORTED, "%s: at most 31 exponents (a 6-bit code)", what);
    if (rows == 0 || K == 0) return QNN_OK;
    QNN_REQUIRE(x && out, QNN_ERR_INVALID_ARG, "%s: NULL pointer", what);
    const int64_t kz = (int64_t)round_up((size_t)K, 32);
    QNN_REQUIRE(ldx >= (transposed ? rows : K) && ld_bytes >= kz, QNN_ERR_INVALID_ARG,
                "%s: ldx below the row length of x, or ld_bytes below K rounded up to 32", what);
    QNN_REQUIRE(aligned(x, 4) && aligned(out, 4) && ld_bytes % 4 == 0, QNN_ERR_ALIGNMENT,
                "%s: pointers and the output row stride must be multiples of 4 bytes", what);
    const int groups = qnn_logquant_groups(emin, emax);
    cudaStream_t st = as_stream(stream);
    if (transposed) {
        QNN_REQUIRE(ceil_div(rows, 32) <= 65535, QNN_ERR_UNSUPPORTED, "%s: too many rows for the launch grid", what);
        const dim3 grid((unsigned)(kz / 32), (unsigned)ceil_div(rows, 32));
        log_groups_t_kernel<<<grid, 256, 0, st>>>(x, rows, K, ldx, emin, emax, groups, static_cast<uint8_t *>(out), ld_bytes);
    } else {
        const int64_t kq = kz / 4;
        const int64_t need = ceil_div(rows * kq, 256), cap = (int64_t)sm_count() * 32;
        const bool vec = (ldx % 4 == 0) && aligned(x, 16);
        log_groups_kernel<<<(int)(need < cap ? need : cap), 256, 0, st>>>(x, rows, K, ldx, emin, emax, groups, static_cast<uint8_t *>(out),
                                                                         ld_bytes, kq, vec);
    }
    return check_launch(what);
}

int qnn_logquant_combine(const int32_t *p, int groups, int64_t M, int64_t N, int64_t ldp, int64_t *out, int64_t ldo, void *stream)
{
    const char *what = "qnn_logquant_combine";
    QNN_REQUIRE(M >= 0 && N >= 0 && groups >= 1 && groups <= 5, QNN_ERR_INVALID_ARG, "%s: bad size or group count", what);
    if (M == 0 || N == 0) return QNN_OK;
    QNN_REQUIRE(p && out, QNN_ERR_INVALID_ARG, "%s: NULL pointer", what);
    QNN_REQUIRE(ldp >= N && ldo >= N, QNN_ERR_INVALID_ARG, "%s: leading dimension below N", what);
    QNN_REQUIRE(aligned(p, 4) && aligned(out, 8), QNN_ERR_ALIGNMENT, "%s: p must be 4-byte, out 8-byte aligned", what);
    const bool vec = N % 4 == 0 && ldp % 4 == 0 && ldo % 2 == 0 && aligned(p, 16) && aligned(out, 16);
    const int64_t need = ceil_div(M * (vec ? N / 4 : N), 256), cap = (int64_t)sm_count() * 32;
    if (vec) log_combine_kernel<true><<<(int)(need < cap ? need : cap), 256, 0, as_stream(stream)>>>(p, groups, M, N, ldp, out, ldo);
    else log_combine_kernel<false><<<(int)(need < cap ? need : cap), 256, 0, as_stream(stream)>>>(p, groups, M, N, ldp, out, ldo);
    return check_launch(what);
}

}  // extern "C"
