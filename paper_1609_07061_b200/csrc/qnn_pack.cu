// Quantise + bit-pack kernels (Eq. 1, Eq. 8, Eq. 9; the 32-per-word
// concatenation of Sec. 6).  All of them are HBM-bound streaming kernels:
// 128-bit coalesced loads, bits assembled with warp shuffles / ballots,
// grids sized from the SM count.
#include "qnn_internal.cuh"

namespace qnn {

// --------------------------------------------------------------------------
// Row-major packing: source [rows, K] -> words [rows, ceil(K/32)].
// A warp owns a (row, chunk) pair; a chunk is 128*UNROLL elements.  Each lane
// loads UNROLL 16-byte vectors (4 elements each), turns each into a nibble and
// the warp ORs the nibbles of 8 neighbouring lanes into one word.  Sources give
// a vector either in one step (nibble) or as a raw load and a later conversion
// (raw, nib_of), which lets a full chunk's loads be issued back to back.
// --------------------------------------------------------------------------

struct SignSrc {
    const float *x;
    int64_t ld;
    static constexpr int kElemBytes = 4;
    __device__ __forceinline__ uint32_t bit(int64_t r, int64_t k) const { return x[r * ld + k] >= 0.0f; }
    __device__ __forceinline__ uint32_t nibble(int64_t r, int64_t k) const
    {
        const float4 v = __ldcs(reinterpret_cast<const float4 *>(x + r * ld + k));
        return (uint32_t)(v.x >= 0.0f) | ((uint32_t)(v.y >= 0.0f) << 1) | ((uint32_t)(v.z >= 0.0f) << 2) |
               ((uint32_t)(v.w >= 0.0f) << 3);
    }
    __device__ __forceinline__ int4 raw(int64_t r, int64_t k) const { return __ldcs(reinterpret_cast<const int4 *>(x + r * ld + k)); }
    __device__ __forceinline__ uint32_t nib_of(const int4 v, int64_t) const
    {
        return (uint32_t)(__int_as_float(v.x) >= 0.0f) | ((uint32_t)(__int_as_float(v.y) >= 0.0f) << 1) | ((uint32_t)(__int_as_float(v.z) >= 0.0f) << 2) | ((uint32_t)(__int_as_float(v.w) >= 0.0f) << 3);
    }
    __host__ bool vector_ok() const { return (ld % 4 == 0) && aligned(x, 16); }
};

struct ThresholdSrc {
    const int32_t *s;
    int64_t ld;
    const int32_t *thr;
    const uint8_t *flip;   // may be null
    __device__ __forceinline__ uint32_t bit(int64_t r, int64_t k) const
    {
        uint32_t b = s[r * ld + k] >= thr[k];
        if (flip) b ^= (uint32_t)(flip[k] != 0);
        return b;
    }
    __device__ __forceinline__ uint32_t nibble(int64_t r, int64_t k) const
    {
        const int4 v = __ldcs(reinterpret_cast<const int4 *>(s + r * ld + k));
        const int4 t = __ldg(reinterpret_cast<const int4 *>(thr + k));
        uint32_t n = (uint32_t)(v.x >= t.x) | ((uint32_t)(v.y >= t.y) << 1) | ((uint32_t)(v.z >= t.z) << 2) |
                     ((uint32_t)(v.w >= t.w) << 3);
        if (flip) {
            const uint32_t f = __ldg(reinterpret_cast<const uint32_t *>(flip + k));   // 4 bytes
            n ^= (uint32_t)((f & 0xffu) != 0) | ((uint32_t)((f & 0xff00u) != 0) << 1) |
                 ((uint32_t)((f & 0xff0000u) != 0) << 2) | ((uint32_t)((f & 0xff000000u) != 0) << 3);
        }
        return n;
    }
    __device__ __forceinline__ int4 raw(int64_t r, int64_t k) const { return __ldcs(reinterpret_cast<const int4 *>(s + r * ld + k)); }
    __device__ __forceinline__ uint32_t nib_of(const int4 v, int64_t k) const
    {
        const int4 t = __ldg(reinterpret_cast<const int4 *>(thr + k));
        uint32_t n = (uint32_t)(v.x >= t.x) | ((uint32_t)(v.y >= t.y) << 1) | ((uint32_t)(v.z >= t.z) << 2) | ((uint32_t)(v.w >= t.w) << 3);
        if (flip) {
            const uint32_t f = __ldg(reinterpret_cast<const uint32_t *>(flip + k));
            n ^= (uint32_t)((f & 0xffu) != 0) | ((uint32_t)((f & 0xff00u) != 0) << 1) | ((uint32_t)((f & 0xff0000u) != 0) << 2) | ((uint32_t)((f & 0xff000000u) != 0) << 3);
        }
        return n;
    }
    __host__ bool vector_ok() const
    {
        return (ld % 4 == 0) && aligned(s, 16) && aligned(thr, 16) && (!flip || aligned(flip, 4));
    }
};

// This HBM-bound kernel lives on the bytes it keeps in flight: a full chunk's UNROLL 16-byte loads are all issued
// before the first one is used (64 registers at four resident blocks per SM hold them).  Measured on B200,
// 10000 x 4096: sign 38.9 -> 30.7 us, threshold 47.1 -> 38.9 us against eight blocks of 32-register threads with
// four loads each; sixteen loads, or three or six blocks, are slower.
template <class Src, int UNROLL, bool VEC>
__global__ void __launch_bounds__(256, 4) row_pack_kernel(Src src, int64_t rows, int64_t K, uint32_t *__restrict__ out,
                                                       int64_t ld_words, int32_t *__restrict__ row_popc,
                                                       int64_t chunks_per_row)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t total = rows * chunks_per_row;
    constexpr int CHUNK = 128 * UNROLL;
    for (int64_t item = warp0; item < total; item += nwarps) {
        const int64_t r = item / chunks_per_row;
        const int64_t k0 = (item - r * chunks_per_row) * CHUNK;
        uint32_t nib[UNROLL];
        if (VEC && k0 + CHUNK <= K) {
            int4 raw[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) raw[u] = src.raw(r, k0 + u * 128 + lane * 4);
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) nib[u] = src.nib_of(raw[u], k0 + u * 128 + lane * 4);
        } else {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int64_t k = k0 + u * 128 + lane * 4;
                uint32_t n = 0;
                if (VEC && k + 4 <= K) {
                    n = src.nibble(r, k);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (k + j < K) n |= src.bit(r, k + j) << j;
                }
                nib[u] = n;
            }
        }
        int pc = 0;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            uint32_t w = nib[u] << (4 * (lane & 7));
            w |= __shfl_xor_sync(0xffffffffu, w, 1);
            w |= __shfl_xor_sync(0xffffffffu, w, 2);
            w |= __shfl_xor_sync(0xffffffffu, w, 4);
            const int64_t k = k0 + u * 128 + (lane >> 3) * 32;   // first element of this lane group's word
            if ((lane & 7) == 0 && k < K) {
                out[r * ld_words + (k >> 5)] = w;
                pc += __popc(w);
            }
        }
        if (row_popc != nullptr) {
            pc += __shfl_xor_sync(0xffffffffu, pc, 8);
            pc += __shfl_xor_sync(0xffffffffu, pc, 16);
            if (lane == 0 && pc) atomicAdd(row_popc + r, pc);
        }
    }
}

template <class Src>
static int launch_row_pack(const Src &src, int64_t rows, int64_t K, uint32_t *out, int64_t ld_words,
                           int32_t *row_popc, cudaStream_t st, const char *what)
{
    if (rows == 0 || K == 0) return QNN_OK;
    if (row_popc) QNN_CUDA(cudaMemsetAsync(row_popc, 0, sizeof(int32_t) * (size_t)rows, st));
    constexpr int UNROLL = 8;
    const int64_t chunks = ceil_div(K, 128 * UNROLL);
    const int64_t warps = rows * chunks;
    const int64_t blocks_needed = ceil_div(warps, 8);
    const int64_t cap = (int64_t)sm_count() * 4;
    const int blocks = (int)(blocks_needed < cap ? blocks_needed : cap);
    if (src.vector_ok())
        row_pack_kernel<Src, UNROLL, true><<<blocks, 256, 0, st>>>(src, rows, K, out, ld_words, row_popc, chunks);
    else
        row_pack_kernel<Src, UNROLL, false><<<blocks, 256, 0, st>>>(src, rows, K, out, ld_words, row_popc, chunks);
    return check_launch(what);
}

// --------------------------------------------------------------------------
// k-bit row-major quantise / plane split.  Lane l of a warp handles elements
// k0 + l + 32*j, so one ballot per plane yields a finished word.
// --------------------------------------------------------------------------

struct KbitF32Src {
    const float *x;
    int64_t ld;
    float lo, hi, inv_step;
    int qmax;
    __device__ __forceinline__ int code(int64_t r, int64_t k) const
    {
        // clip, subtract, multiply, round-half-even: four separately rounded fp32 steps
        float t = __ldcs(x + r * ld + k);
        t = fminf(fmaxf(t, lo), hi);               // NaN -> lo
        const float d = __fsub_rn(t, lo);
        const float u = __fmul_rn(d, inv_step);
        int q = __float2int_rn(u);
        q = q < 0 ? 0 : (q > qmax ? qmax : q);
        return q;
    }
};

struct U8Src {
    const uint8_t *x;
    int64_t ld;
    int qmask;
    __device__ __forceinline__ int code(int64_t r, int64_t k) const { return (int)x[r * ld + k] & qmask; }
};

template <class Src>
__global__ void __launch_bounds__(256) row_planes_kernel(Src src, int64_t rows, int64_t K, int bits,
                                                         uint32_t *__restrict__ planes, int64_t ld_words,
                                                         int64_t plane_stride, int32_t *__restrict__ row_sum,
                                                         int64_t chunks_per_row)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t total = rows * chunks_per_row;
    constexpr int WORDS = 4;                       // words per plane per warp item
    for (int64_t item = warp0; item < total; item += nwarps) {
        const int64_t r = item / chunks_per_row;
        const int64_t k0 = (item - r * chunks_per_row) * (32 * WORDS);
        int q[WORDS];
        int sum = 0;
#pragma unroll
        for (int j = 0; j < WORDS; ++j) {
            const int64_t k = k0 + 32 * j + lane;
            q[j] = (k < K) ? src.code(r, k) : 0;
            sum += q[j];
        }
#pragma unroll
        for (int j = 0; j < WORDS; ++j) {
            const int64_t kw = (k0 >> 5) + j;
            const bool live = (k0 + 32 * j) < K;   // warp-uniform
            for (int i = 0; i < bits; ++i) {
                const uint32_t w = __ballot_sync(0xffffffffu, (q[j] >> i) & 1);
                if (live && lane == i) planes[i * plane_stride + r * ld_words + kw] = w;
            }
        }
        if (row_sum != nullptr) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0 && sum) atomicAdd(row_sum + r, sum);
        }
    }
}

// uint8 codes, vector path (K and the row pitch multiples of 16, 16-byte aligned base): a lane loads 16
// consecutive codes at once; bit i of every byte is gathered with one multiply per four codes
// (0x01020408 moves the four byte-LSBs into one nibble), two neighbouring lanes make a 32-bit word.
__global__ void __launch_bounds__(256) row_planes_u8_vec_kernel(const uint8_t *__restrict__ x, int64_t ld, int qmask,
                                                                int64_t rows, int64_t K, int bits,
                                                                uint32_t *__restrict__ planes, int64_t ld_words,
                                                                int64_t plane_stride, int32_t *__restrict__ row_sum,
                                                                int64_t chunks_per_row)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t total = rows * chunks_per_row;
    const uint32_t qm4 = (uint32_t)qmask * 0x01010101u;
    for (int64_t item = warp0; item < total; item += nwarps) {
        const int64_t r = item / chunks_per_row;
        const int64_t k0 = (item - r * chunks_per_row) * 512;
        const int64_t k = k0 + lane * 16;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (k < K) v = __ldcs(reinterpret_cast<const uint4 *>(x + r * ld + k));
        v.x &= qm4; v.y &= qm4; v.z &= qm4; v.w &= qm4;
        const int64_t kw = (k0 >> 5) + (lane >> 1);
        const bool store = ((lane & 1) == 0) && (k < K);       // K is a multiple of 16: an even lane's word holds at least 16 codes
        for (int i = 0; i < bits; ++i) {
            const uint32_t h = ((((v.x >> i) & 0x01010101u) * 0x01020408u) >> 24) |
                               (((((v.y >> i) & 0x01010101u) * 0x01020408u) >> 24) << 4) |
                               (((((v.z >> i) & 0x01010101u) * 0x01020408u) >> 24) << 8) |
                               (((((v.w >> i) & 0x01010101u) * 0x01020408u) >> 24) << 12);
            const uint32_t other = __shfl_xor_sync(0xffffffffu, h, 1);
            if (store) planes[i * plane_stride + r * ld_words + kw] = h | (other << 16);
        }
        if (row_sum != nullptr) {
            int sum = __dp4a(v.x, 0x01010101u, 0u) + __dp4a(v.y, 0x01010101u, 0u) + __dp4a(v.z, 0x01010101u, 0u) +
                      __dp4a(v.w, 0x01010101u, 0u);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
            if (lane == 0 && sum) atomicAdd(row_sum + r, sum);
        }
    }
}

template <class Src>
static int launch_row_planes(const Src &src, int64_t rows, int64_t K, int bits, uint32_t *planes, int64_t ld_words,
                             int64_t plane_stride, int32_t *row_sum, cudaStream_t st, const char *what)
{
    if (rows == 0 || K == 0) return QNN_OK;
    if (row_sum) QNN_CUDA(cudaMemsetAsync(row_sum, 0, sizeof(int32_t) * (size_t)rows, st));
    const int64_t chunks = ceil_div(K, 128);
    const int64_t blocks_needed = ceil_div(rows * chunks, 8);
    const int64_t cap = (int64_t)sm_count() * 8;
    const int blocks = (int)(blocks_needed < cap ? blocks_needed : cap);
    row_planes_kernel<Src><<<blocks, 256, 0, st>>>(src, rows, K, bits, planes, ld_words, plane_stride, row_sum, chunks);
    return check_launch(what);
}

// --------------------------------------------------------------------------
// Transposed packing: source [batch][K, N] (row-major, K strided) -> words
// [batch][N, ld_words] packed along K.  A thread owns 4 neighbouring n and
// KW consecutive words of K (32*KW source rows): every load is a 16-byte
// vector along n, coalesced across the warp; no shuffles are needed because a
// thread sees all 32 rows of its words.
// --------------------------------------------------------------------------

struct SignCode {
    __device__ __forceinline__ int operator()(float v) const { return v >= 0.0f; }
};
struct KbitCode {
    float lo, hi, inv_step;
    int qmax;
    __device__ __forceinline__ int operator()(float t) const
    {
        t = fminf(fmaxf(t, lo), hi);
        const float d = __fsub_rn(t, lo);
        const float u = __fmul_rn(d, inv_step);
        int q = __float2int_rn(u);
        return q < 0 ? 0 : (q > qmax ? qmax : q);
    }
};

template <class Code, int NB /*planes*/, bool VEC>
__global__ void __launch_bounds__(128) trans_pack_kernel(const float *__restrict__ w, int64_t K, int64_t N, int64_t ldw,
                                                         int64_t batch_stride_in, Code code,
                                                         uint32_t *__restrict__ out, int64_t ld_words,
                                                         int64_t plane_stride, int64_t batch_stride_out,
                                                         int32_t *__restrict__ row_sum)
{
    // grid: x over n (128 threads * 4 n), y over words of K, z over batch
    const int64_t n0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    const int64_t kw = blockIdx.y;
    const int64_t bz = blockIdx.z;
    if (n0 >= N) return;
    const float *src = w + bz * batch_stride_in;
    uint32_t word[NB][4];
#pragma unroll
    for (int p = 0; p < NB; ++p)
#pragma unroll
        for (int c = 0; c < 4; ++c) word[p][c] = 0;
    int sum[4] = {0, 0, 0, 0};
    const int64_t kbase = kw * 32;
    if (VEC && n0 + 4 <= N && kbase + 32 <= K) {
        // whole word, whole vectors: sixteen loads issued before the first is converted, twice (measured on B200,
        // 4096 x 4096: 26.6 -> 18.4 us; the unrolled loop below keeps only a few loads in flight)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float4 t[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) t[j] = __ldcs(reinterpret_cast<const float4 *>(src + (kbase + h * 16 + j) * ldw + n0));
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float v[4] = {t[j].x, t[j].y, t[j].z, t[j].w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int q = code(v[c]);
                    sum[c] += q;
#pragma unroll
                    for (int p = 0; p < NB; ++p) word[p][c] |= (uint32_t)((q >> p) & 1) << (h * 16 + j);
                }
            }
        }
    } else
#pragma unroll 8
    for (int j = 0; j < 32; ++j) {
        const int64_t k = kbase + j;
        if (k < K) {
            float v[4];
            if (VEC && n0 + 4 <= N) {
                const float4 t = __ldcs(reinterpret_cast<const float4 *>(src + k * ldw + n0));
                v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) v[c] = (n0 + c < N) ? src[k * ldw + n0 + c] : -1.0f;
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int q = code(v[c]);
                sum[c] += q;
#pragma unroll
                for (int p = 0; p < NB; ++p) word[p][c] |= (uint32_t)((q >> p) & 1) << j;
            }
        }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        if (n0 + c < N) {
#pragma unroll
            for (int p = 0; p < NB; ++p)
                out[bz * batch_stride_out + p * plane_stride + (n0 + c) * ld_words + kw] = word[p][c];
            if (row_sum != nullptr && sum[c]) atomicAdd(row_sum + n0 + c, sum[c]);
        }
    }
}

template <class Code, int NB>
static int launch_trans_pack_nb(const float *w, int64_t K, int64_t N, int64_t ldw, int64_t batch, int64_t bs_in,
                                const Code &code, uint32_t *out, int64_t ld_words, int64_t plane_stride,
                                int64_t bs_out, int32_t *row_sum, cudaStream_t st, const char *what)
{
    if (K == 0 || N == 0 || batch == 0) return QNN_OK;
    if (row_sum) QNN_CUDA(cudaMemsetAsync(row_sum, 0, sizeof(int32_t) * (size_t)N, st));
    const int64_t kwords = ceil_div(K, 32);
    QNN_REQUIRE(kwords <= 65535 && batch <= 65535, QNN_ERR_UNSUPPORTED, "%s: K/32 or batch exceeds 65535", what);
    dim3 grid((unsigned)ceil_div(N, 128 * 4), (unsigned)kwords, (unsigned)batch);
    const bool vec = (ldw % 4 == 0) && (bs_in % 4 == 0) && aligned(w, 16);
    if (vec)
        trans_pack_kernel<Code, NB, true><<<grid, 128, 0, st>>>(w, K, N, ldw, bs_in, code, out, ld_words, plane_stride,
                                                                bs_out, row_sum);
    else
        trans_pack_kernel<Code, NB, false><<<grid, 128, 0, st>>>(w, K, N, ldw, bs_in, code, out, ld_words, plane_stride,
                                                                 bs_out, row_sum);
    return check_launch(what);
}

// --------------------------------------------------------------------------
// Logarithmic quantiser (Eq. 10): AP2(x) = sign(x) * 2^round(log2|x|) with the
// magnitude clipped to [2^emin, 2^emax], written as the int8 value
// sign * 2^(e - emin) -- directly an operand of the int8 tensor-core form.
// round(log2|x|) comes from the float's own fields: the exponent, plus one when
// the mantissa is above the largest float below sqrt(2) (sqrt(2) is not a
// float, so there are no ties).  Zero and denormals clip to emin, infinities
// and NaN to emax; the sign is Eq. 1's (x >= 0 gives +1, NaN gives -1).
// --------------------------------------------------------------------------
__device__ __forceinline__ uint32_t logquant_byte(float x, int emin, int emax)
{
    const uint32_t a = __float_as_uint(x) & 0x7fffffffu;
    int e;
    if (a >= 0x7f800000u) e = emax;
    else if (a < 0x00800000u) e = emin;
    else {
        e = (int)(a >> 23) - 127 + (int)((a & 0x7fffffu) > 0x3504f3u);
        e = e < emin ? emin : (e > emax ? emax : e);
    }
    const int v = 1 << (e - emin);
    return (uint32_t)(x >= 0.0f ? v : -v) & 0xffu;
}

// One thread per 4 consecutive elements of a row (kq = ceil(Kz / 4) groups per row, Kz = K rounded up to 32: the
// bytes between K and Kz are written as zero so that the row is a valid tensor-core operand).
__global__ void __launch_bounds__(256) logquant_i8_kernel(const float *__restrict__ x, int64_t rows, int64_t K, int64_t ldx,
                                                          int emin, int emax, uint8_t *__restrict__ out, int64_t ld_bytes,
                                                          int64_t kq, bool vec)
{
    const int64_t total = rows * kq;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / kq, k = (i - r * kq) * 4;
        uint32_t w = 0;
        if (vec && k + 4 <= K) {
            const float4 v = __ldcs(reinterpret_cast<const float4 *>(x + r * ldx + k));
            w = logquant_byte(v.x, emin, emax) | (logquant_byte(v.y, emin, emax) << 8) | (logquant_byte(v.z, emin, emax) << 16) |
                (logquant_byte(v.w, emin, emax) << 24);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (k + j < K) w |= logquant_byte(x[r * ldx + k + j], emin, emax) << (8 * j);
        }
        *reinterpret_cast<uint32_t *>(out + r * ld_bytes + k) = w;
    }
}

}  // namespace qnn

using namespace qnn;

extern "C" {

int qnn_quantize_pack_sign(const float *x, int64_t rows, int64_t K, int64_t ldx, uint32_t *out, int64_t ld_words,
                           int32_t *row_popc, void *stream)
{
    QNN_REQUIRE(rows >= 0 && K >= 0, QNN_ERR_INVALID_ARG, "qnn_quantize_pack_sign: negative size");
    if (rows == 0 || K == 0) return QNN_OK;
    QNN_REQUIRE(x && out, QNN_ERR_INVALID_ARG, "qnn_quantize_pack_sign: NULL pointer");
    QNN_REQUIRE(ldx >= K && ld_words >= ceil_div(K, 32), QNN_ERR_INVALID_ARG,
                "qnn_quantize_pack_sign: leading dimension too small");
    QNN_REQUIRE(aligned(x, 4) && aligned(out, 4) && (!row_popc || aligned(row_popc, 4)), QNN_ERR_ALIGNMENT,
                "qnn_quantize_pack_sign: pointers must be 4-byte aligned");
    SignSrc src{x, ldx};
    return launch_row_pack(src, rows, K, out, ld_words, row_popc, as_stream(stream), "qnn_quantize_pack_sign");
}

int qnn_threshold_pack(const int32_t *s, int64_t M, int64_t N, int64_t lds, const int32_t *thr, const uint8_t *flip,
                       uint32_t *out, int64_t ld_words, void *stream)
{
    QNN_REQUIRE(M >= 0 && N >= 0, QNN_ERR_INVALID_ARG, "qnn_threshold_pack: negative size");
    if (M == 0 || N == 0) return QNN_OK;
    QNN_REQUIRE(s && thr && out, QNN_ERR_INVALID_ARG, "qnn_threshold_pack: NULL pointer");
    QNN_REQUIRE(lds >= N && ld_words >= ceil_div(N, 32), QNN_ERR_INVALID_ARG,
                "qnn_threshold_pack: leading dimension too small");
    QNN_REQUIRE(aligned(s, 4) && aligned(thr, 4) && aligned(out, 4), QNN_ERR_ALIGNMENT,
                "qnn_threshold_pack: pointers must be 4-byte aligned");
    ThresholdSrc src{s, lds, thr, flip};
    return launch_row_pack(src, M, N, out, ld_words, nullptr, as_stream(stream), "qnn_threshold_pack");
}

static int check_kbit(const char *what, int bits, float lo, float hi)
{
    QNN_REQUIRE(bits >= 1 && bits <= 8, QNN_ERR_INVALID_ARG, "%s: bits must be in 1..8", what);
    QNN_REQUIRE(hi > lo, QNN_ERR_INVALID_ARG, "%s: need hi > lo", what);
    return QNN_OK;
}

int qnn_quantize_pack_kbit(const float *x, int64_t rows, int64_t K, int64_t ldx, int bits, float lo, float hi,
                           uint32_t *planes, int64_t ld_words, int64_t plane_stride_words, int32_t *row_sum_q,
                           void *stream)
{
    QNN_REQUIRE(rows >= 0 && K >= 0, QNN_ERR_INVALID_ARG, "qnn_quantize_pack_kbit: negative size");
    if (int rc = check_kbit("qnn_quantize_pack_kbit", bits, lo, hi)) return rc;
    if (rows == 0 || K == 0) return QNN_OK;
    QNN_REQUIRE(x && planes, QNN_ERR_INVALID_ARG, "qnn_quantize_pack_kbit: NULL pointer");
    QNN_REQUIRE(ldx >= K && ld_words >= ceil_div(K, 32) && (bits == 1 || plane_stride_words >= rows * ld_words),
                QNN_ERR_INVALID_ARG, "qnn_quantize_pack_kbit: leading dimension or plane stride too small");
    const float inv_step = (float)((1 << bits) - 1) / (hi - lo);
    KbitF32Src src{x, ldx, lo, hi, inv_step, (1 << bits) - 1};
    return launch_row_planes(src, rows, K, bits, planes, ld_words, plane_stride_words, row_sum_q, as_stream(stream),
                             "qnn_quantize_pack_kbit");
}

int qnn_pack_planes_u8(const uint8_t *x, int64_t rows, int64_t K, int64_t ldx, int bits, uint32_t *planes,
                       int64_t ld_words, int64_t plane_stride_words, int32_t *row_sum_q, void *stream)
{
    QNN_REQUIRE(rows >= 0 && K >= 0, QNN_ERR_INVALID_ARG, "qnn_pack_planes_u8: negative size");
    QNN_REQUIRE(bits >= 1 && bits <= 8, QNN_ERR_INVALID_ARG, "qnn_pack_planes_u8: bits must be in 1..8");
    if (rows == 0 || K == 0) return QNN_OK;
    QNN_REQUIRE(x && planes, QNN_ERR_INVALID_ARG, "qnn_pack_planes_u8: NULL pointer");
    QNN_REQUIRE(ldx >= K && ld_words >= ceil_div(K, 32) && (bits == 1 || plane_stride_words >= rows * ld_words),
                QNN_ERR_INVALID_ARG, "qnn_pack_planes_u8: leading dimension or plane stride too small");
    cudaStream_t st = as_stream(stream);
    if (K % 16 == 0 && ldx % 16 == 0 && aligned(x, 16)) {
        if (row_sum_q) QNN_CUDA(cudaMemsetAsync(row_sum_q, 0, sizeof(int32_t) * (size_t)rows, st));
        const int64_t chunks = ceil_div(K, 512);
        const int64_t blocks_needed = ceil_div(rows * chunks, 8);
        const int64_t cap = (int64_t)sm_count() * 8;
        const int blocks = (int)(blocks_needed < cap ? blocks_needed : cap);
        row_planes_u8_vec_kernel<<<blocks, 256, 0, st>>>(x, ldx, (1 << bits) - 1, rows, K, bits, planes, ld_words,
                                                         plane_stride_words, row_sum_q, chunks);
        return check_launch("qnn_pack_planes_u8");
    }
    U8Src src{x, ldx, (1 << bits) - 1};
    return launch_row_planes(src, rows, K, bits, planes, ld_words, plane_stride_words, row_sum_q, st, "qnn_pack_planes_u8");
}

int qnn_quantize_pack_sign_t(const float *w, int64_t K, int64_t N, int64_t ldw, uint32_t *out, int64_t ld_words,
                             int32_t *row_popc, void *stream)
{
    QNN_REQUIRE(K >= 0 && N >= 0, QNN_ERR_INVALID_ARG, "qnn_quantize_pack_sign_t: negative size");
    if (K == 0 || N == 0) return QNN_OK;
    QNN_REQUIRE(w && out, QNN_ERR_INVALID_ARG, "qnn_quantize_pack_sign_t: NULL pointer");
    QNN_REQUIRE(ldw >= N && ld_words >= ceil_div(K, 32), QNN_ERR_INVALID_ARG,
                "qnn_quantize_pack_sign_t: leading dimension too small");
    return launch_trans_pack_nb<SignCode, 1>(w, K, N, ldw, 1, 0, SignCode{}, out, ld_words, 0, 0, row_popc,
                                             as_stream(stream), "qnn_quantize_pack_sign_t");
}

int qnn_quantize_pack_sign_nchw(const float *x, int B, int C, int H, int W, uint32_t *out, void *stream)
{
    QNN_REQUIRE(B >= 0 && C >= 0 && H >= 0 && W >= 0, QNN_ERR_INVALID_ARG, "qnn_quantize_pack_sign_nchw: negative size");
    if (B == 0 || C == 0 || H == 0 || W == 0) return QNN_OK;
    QNN_REQUIRE(x && out, QNN_ERR_INVALID_ARG, "qnn_quantize_pack_sign_nchw: NULL pointer");
    // per image: a [C, H*W] matrix packed along C for every pixel
    const int64_t hw = (int64_t)H * W;
    const int64_t cw = ceil_div(C, 32);
    return launch_trans_pack_nb<SignCode, 1>(x, C, hw, hw, B, (int64_t)C * hw, SignCode{}, out, cw, 0, hw * cw, nullptr,
                                             as_stream(stream), "qnn_quantize_pack_sign_nchw");
}

int qnn_quantize_pack_kbit_t(const float *w, int64_t K, int64_t N, int64_t ldw, int bits, float lo, float hi,
                             uint32_t *planes, int64_t ld_words, int64_t plane_stride_words, int32_t *row_sum_q,
                             void *stream)
{
    QNN_REQUIRE(K >= 0 && N >= 0, QNN_ERR_INVALID_ARG, "qnn_quantize_pack_kbit_t: negative size");
    if (int rc = check_kbit("qnn_quantize_pack_kbit_t", bits, lo, hi)) return rc;
    if (K == 0 || N == 0) return QNN_OK;
    QNN_REQUIRE(w && planes, QNN_ERR_INVALID_ARG, "qnn_quantize_pack_kbit_t: NULL pointer");
    QNN_REQUIRE(ldw >= N && ld_words >= ceil_div(K, 32) && (bits == 1 || plane_stride_words >= N * ld_words),
                QNN_ERR_INVALID_ARG, "qnn_quantize_pack_kbit_t: leading dimension or plane stride too small");
    const float inv_step = (float)((1 << bits) - 1) / (hi - lo);
    KbitCode code{lo, hi, inv_step, (1 << bits) - 1};
    cudaStream_t st = as_stream(stream);
    const char *what = "qnn_quantize_pack_kbit_t";
    switch (bits) {
        case 1: return launch_trans_pack_nb<KbitCode, 1>(w, K, N, ldw, 1, 0, code, planes, ld_words, plane_stride_words, 0, row_sum_q, st, what);
        case 2: return launch_trans_pack_nb<KbitCode, 2>(w, K, N, ldw, 1, 0, code, planes, ld_words, plane_stride_words, 0, row_sum_q, st, what);
        case 3: return launch_trans_pack_nb<KbitCode, 3>(w, K, N, ldw, 1, 0, code, planes, ld_words, plane_stride_words, 0, row_sum_q, st, what);
        case 4: return launch_trans_pack_nb<KbitCode, 4>(w, K, N, ldw, 1, 0, code, planes, ld_words, plane_stride_words, 0, row_sum_q, st, what);
        case 5: return launch_trans_pack_nb<KbitCode, 5>(w, K, N, ldw, 1, 0, code, planes, ld_words, plane_stride_words, 0, row_sum_q, st, what);
        case 6: return launch_trans_pack_nb<KbitCode, 6>(w, K, N, ldw, 1, 0, code, planes, ld_words, plane_stride_words, 0, row_sum_q, st, what);
        case 7: return launch_trans_pack_nb<KbitCode, 7>(w, K, N, ldw, 1, 0, code, planes, ld_words, plane_stride_words, 0, row_sum_q, st, what);
        default: return launch_trans_pack_nb<KbitCode, 8>(w, K, N, ldw, 1, 0, code, planes, ld_words, plane_stride_words, 0, row_sum_q, st, what);
    }
}

int qnn_logquant_pack_i8(const float *x, int64_t rows, int64_t K, int64_t ldx, int emin, int emax, void *out, int64_t ld_bytes,
                         void *stream)
{
    QNN_REQUIRE(rows >= 0 && K >= 0, QNN_ERR_INVALID_ARG, "qnn_logquant_pack_i8: negative size");
    QNN_REQUIRE(emax >= emin && emin >= -126 && emax <= 127, QNN_ERR_INVALID_ARG,
                "qnn_logquant_pack_i8: need -126 <= emin <= emax <= 127");
    QNN_REQUIRE(emax - emin <= 6, QNN_ERR_UNSUPPORTED, "qnn_logquant_pack_i8: at most 7 levels (2^6 = 64) fit an int8 value");
    if (rows == 0 || K == 0) return QNN_OK;
    QNN_REQUIRE(x && out, QNN_ERR_INVALID_ARG, "qnn_logquant_pack_i8: NULL pointer");
    const int64_t kz = (int64_t)round_up((size_t)K, 32);
    QNN_REQUIRE(ldx >= K && ld_bytes >= kz, QNN_ERR_INVALID_ARG,
                "qnn_logquant_pack_i8: ldx below K, or ld_bytes below K rounded up to 32");
    QNN_REQUIRE(aligned(x, 4) && aligned(out, 4) && ld_bytes % 4 == 0, QNN_ERR_ALIGNMENT,
                "qnn_logquant_pack_i8: pointers and the output row stride must be multiples of 4 bytes");
    const int64_t kq = kz / 4;
    const bool vec = (ldx % 4 == 0) && aligned(x, 16);
    const int64_t need = ceil_div(rows * kq, 256), cap = (int64_t)sm_count() * 8;
    logquant_i8_kernel<<<(int)(need < cap ? need : cap), 256, 0, as_stream(stream)>>>(x, rows, K, ldx, emin, emax,
                                                                                     static_cast<uint8_t *>(out), ld_bytes, kq, vec);
    return check_launch("qnn_logquant_pack_i8");
}

}  // extern "C"
