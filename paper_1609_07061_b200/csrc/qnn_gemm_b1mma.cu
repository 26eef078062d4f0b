// Legacy tensor-core path for the 1-bit x 1-bit product: mma.sync m16n8k256 on
// b1 operands with xor + popc accumulation, fed from cp.async-staged shared
// tiles.  Kept as a measured competitor of the CUDA-core and tcgen05 paths.
#include "qnn_internal.cuh"

namespace qnn {
namespace {

constexpr int B1_BM = 128, B1_BN = 128;
constexpr int B1_KW = 16;             // words of K per stage (two k256 steps)
constexpr int B1_LD = B1_KW + 4;      // padded row stride in words: conflict-free fragment loads
constexpr int B1_THREADS = 256;

struct B1Params {
    GemmArgs g;
    int64_t kwords;
    int32_t kconst;                   // K (true number of products)
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

__device__ __forceinline__ void mma_b1_xor(int (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2])
{
    asm volatile(
        "mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};\n"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// rows x B1_KW words of one operand tile -> shared [rows][B1_LD]; 16-byte chunks, zero-filled outside the matrix
__device__ __forceinline__ void b1_load_tile(uint32_t smem_base, const uint32_t *__restrict__ src, int64_t ld, int64_t row0,
                                             int64_t nrows, int64_t kw0, int64_t kwords, int tid)
{
    constexpr int CHUNKS = B1_KW / 4;
    for (int e = tid; e < 128 * CHUNKS; e += B1_THREADS) {
        const int ch = e % CHUNKS;
        const int row = e / CHUNKS;
        const int64_t gr = row0 + row;
        const int64_t gk = kw0 + ch * 4;
        int bytes = 0;
        if (gr < nrows && gk < kwords) {
            const int64_t left = kwords - gk;
            bytes = left >= 4 ? 16 : (int)left * 4;
        }
        const uint32_t *gp = bytes ? (src + gr * ld + gk) : src;
        cp_async16(smem_base + 4u * (uint32_t)(row * B1_LD + ch * 4), gp, bytes);
    }
}

__global__ void __launch_bounds__(B1_THREADS) gemm_b1_kernel(const B1Params P)
{
    __shared__ __align__(16) uint32_t sm[2][2][128 * B1_LD];      // [stage][A|B][rows * stride]
    const GemmArgs &g = P.g;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm = warp >> 2, wn = warp & 3;                      // 2 x 4 warps, warp tile 64 x 32
    const int gq = lane >> 2, tq = lane & 3;
    const int64_t m0 = (int64_t)blockIdx.y * B1_BM, n0 = (int64_t)blockIdx.x * B1_BN;

    int acc[4][4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[i][j][r] = 0;

    const int64_t ktiles = (P.kwords + B1_KW - 1) / B1_KW;
    auto issue = [&](int64_t kt, int st) {
        b1_load_tile((uint32_t)__cvta_generic_to_shared(&sm[st][0][0]), g.a, g.lda, m0, g.M, kt * B1_KW, P.kwords, tid);
        b1_load_tile((uint32_t)__cvta_generic_to_shared(&sm[st][1][0]), g.b, g.ldb, n0, g.N, kt * B1_KW, P.kwords, tid);
        asm volatile("cp.async.commit_group;\n" ::: "memory");
    };
    if (ktiles > 0) issue(0, 0);
    for (int64_t kt = 0; kt < ktiles; ++kt) {
        const int st = (int)(kt & 1);
        if (kt + 1 < ktiles) {
            issue(kt + 1, st ^ 1);
            asm volatile("cp.async.wait_group 1;\n" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;\n" ::: "memory");
        }
        __syncthreads();
        const uint32_t *As = &sm[st][0][0];
        const uint32_t *Bs = &sm[st][1][0];
#pragma unroll
        for (int ks = 0; ks < B1_KW / 8; ++ks) {
            uint32_t bf[4][2];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t *bp = Bs + (wn * 32 + j * 8 + gq) * B1_LD + ks * 8 + tq;
                bf[j][0] = bp[0];
                bf[j][1] = bp[4];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t af[4];
                const uint32_t *ap = As + (wm * 64 + i * 16 + gq) * B1_LD + ks * 8 + tq;
                af[0] = ap[0];
                af[1] = ap[8 * B1_LD];
                af[2] = ap[4];
                af[3] = ap[8 * B1_LD + 4];
#pragma unroll
                for (int j = 0; j < 4; ++j) mma_b1_xor(acc[i][j], af, bf[j]);
            }
        }
        __syncthreads();
    }

    // epilogue: thread owns rows (gq, gq+8) of each 16-row tile and columns 2*tq, 2*tq+1 of each 8-column tile
    const bool want_bits = g.out_bits != nullptr, want_int = g.out != nullptr;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int64_t m = m0 + wm * 64 + i * 16 + gq + 8 * h;
            const bool mrow = m < g.M;
            uint32_t byte = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int64_t n = n0 + wn * 32 + j * 8 + 2 * tq + e;
                    const int32_t val = P.kconst - 2 * acc[i][j][2 * h + e];
                    if (mrow && n < g.N) {
                        if (want_int) {
                            if (g.epilogue == EPI_NCHW) {
                                const int64_t img = m / g.hw, pix = m - img * g.hw;
                                g.out[(img * g.N + n) * g.hw + pix] = val;
                            } else {
                                g.out[m * g.ldo + n] = val;
                            }
                        }
                        if (want_bits) {
                            uint32_t b = val >= __ldg(g.thr + n);
                            if (g.flip) b ^= (uint32_t)(__ldg(g.flip + n) != 0);
                            byte |= b << (j * 8 + 2 * tq + e);
                        }
                    }
                }
            }
            if (want_bits) {
                byte |= __shfl_xor_sync(0xffffffffu, byte, 1);
                byte |= __shfl_xor_sync(0xffffffffu, byte, 2);
                const int64_t nw = n0 + wn * 32;
                if (tq == 0 && mrow && nw < g.N) g.out_bits[m * g.ld_bits + (nw >> 5)] = byte;
            }
        }
    }
}

}  // namespace

int launch_gemm_b1mma(const GemmArgs &g, cudaStream_t st)
{
    QNN_REQUIRE(g.ka == 1 && g.kb == 1 && g.a_mode == QNN_MODE_PM1 && g.b_mode == QNN_MODE_PM1, QNN_ERR_UNSUPPORTED,
                "b1 mma path handles the 1-bit x 1-bit +-1 product only");
    QNN_REQUIRE(g.lda % 4 == 0 && g.ldb % 4 == 0 && aligned(g.a, 16) && aligned(g.b, 16), QNN_ERR_UNSUPPORTED,
                "b1 mma path needs 16-byte aligned operands and leading dimensions that are multiples of 4 words");
    if (g.M == 0 || g.N == 0) return QNN_OK;
    B1Params P;
    P.g = g;
    P.kwords = g.kwords > 0 ? g.kwords : ceil_div(g.K, 32);
    P.kconst = (int32_t)g.K;
    const int64_t gy = ceil_div(g.M, B1_BM);
    QNN_REQUIRE(gy <= 65535, QNN_ERR_UNSUPPORTED, "b1 mma path: M too large for the launch grid");
    dim3 grid((unsigned)ceil_div(g.N, B1_BN), (unsigned)gy);
    profile_before(st);
    gemm_b1_kernel<<<grid, B1_THREADS, 0, st>>>(P);
    profile_after(st);
    return check_launch("b1 mma gemm");
}

}  // namespace qnn
