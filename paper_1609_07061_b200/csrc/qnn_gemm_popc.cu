// CUDA-core matrix product on packed bits: Eq. 11 as written (xor / and,
// popc, accumulate), register-tiled, with packed tiles staged through shared
// memory by cp.async in a two-stage pipeline.  Handles every shape, plane
// count and mode; the tensor-core paths are measured against it.
//
// Per plane pair (i, j) the kernel accumulates 2^(i+j) * popc(a_i OP b_j):
//   PM1 x PM1 : OP = xor, out = K*La*Lb - 2*acc            (La = 2^ka - 1)
//   U01 x PM1 : OP = and, out = 2*acc - Lb * sum_k qa[m,k]
//   PM1 x U01 : OP = and, out = 2*acc - La * sum_k qb[n,k]
//   U01 x U01 : OP = and, out = acc
// Pad bits are zero in both operands, so they add nothing to either popc.
#include "qnn_internal.cuh"

namespace qnn {

namespace {

constexpr int KT = 8;        // 32-bit words of K per pipeline stage (one 32-byte sector per row)
constexpr int PADW = 4;      // row padding of the transposed shared tiles (keeps 16-byte alignment)
constexpr int THREADS = 256;

enum Mode { M_XOR = 0, M_AND_SA = 1, M_AND_SB = 2, M_AND = 3 };

struct PopcParams {
    GemmArgs g;
    int64_t kwords;          // ceil(K/32)
    int32_t kll;             // K * La * Lb (M_XOR)
    int32_t la, lb;
};

__device__ __forceinline__ void cp_async4(uint32_t smem_addr, const void *gptr, bool valid)
{
    const int sz = valid ? 4 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(smem_addr), "l"(gptr), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

// Stage loader: words [planes][rows of this tile][KT] -> shared [plane][kw][rows + PADW].
template <int ROWS>
__device__ __forceinline__ void load_tile(uint32_t smem_base, const uint32_t *__restrict__ src, int planes,
                                          int64_t plane_stride, int64_t ld, int64_t row0, int64_t nrows, int64_t kw0,
                                          int64_t kwords, int tid)
{
    const int total = planes * ROWS * KT;
    for (int e = tid; e < total; e += THREADS) {
        const int kw = e % KT;
        const int row = (e / KT) % ROWS;
        const int p = e / (KT * ROWS);
        const int64_t gr = row0 + row;
        const int64_t gk = kw0 + kw;
        const bool valid = (gr < nrows) && (gk < kwords);
        const uint32_t *gp = valid ? (src + p * plane_stride + gr * ld + gk) : src;
        const uint32_t dst = smem_base + 4u * (uint32_t)((p * KT + kw) * (ROWS + PADW) + row);
        cp_async4(dst, gp, valid);
    }
}

template <int BM, int BN, int TM, int TN, int MODE, bool SINGLE>
__global__ void __launch_bounds__(THREADS) gemm_popc_kernel(const PopcParams P)
{
    static_assert((BM / TM) * (BN / TN) == THREADS, "tile / thread mismatch");
    static_assert(BN / TN == 16, "epilogue assumes 16 threads across N");
    static_assert(TM % 4 == 0 && TN % 4 == 0, "fragments are 128-bit");
    constexpr int G = TN / 4;                 // column groups of 4 per thread
    constexpr int GSTRIDE = BN / G;           // distance between a thread's column groups
    extern __shared__ __align__(16) uint32_t smem[];

    const GemmArgs &g = P.g;
    const int ka = SINGLE ? 1 : g.ka;
    const int kb = SINGLE ? 1 : g.kb;
    const int tid = threadIdx.x;
    const int tx = tid & 15;
    const int ty = tid >> 4;
    const int64_t m0 = (int64_t)blockIdx.y * BM;
    const int64_t n0 = (int64_t)blockIdx.x * BN;

    const int a_stage_words = ka * KT * (BM + PADW);
    const int b_stage_words = kb * KT * (BN + PADW);
    const int stage_words = a_stage_words + b_stage_words;
    const uint32_t smem_u32 = (uint32_t)__cvta_generic_to_shared(smem);

    int32_t acc[TM][TN];
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < TN; ++c) acc[r][c] = 0;
    int32_t sa[TM], sb[TN];
#pragma unroll
    for (int r = 0; r < TM; ++r) sa[r] = 0;
#pragma unroll
    for (int c = 0; c < TN; ++c) sb[c] = 0;

    const int64_t ktiles = (P.kwords + KT - 1) / KT;

    auto issue = [&](int64_t kt, int stage) {
        const uint32_t base = smem_u32 + 4u * (uint32_t)(stage * stage_words);
        load_tile<BM>(base, g.a, ka, g.a_plane_stride, g.lda, m0, g.M, kt * KT, P.kwords, tid);
        load_tile<BN>(base + 4u * (uint32_t)a_stage_words, g.b, kb, g.b_plane_stride, g.ldb, n0, g.N, kt * KT,
                      P.kwords, tid);
        cp_async_commit();
    };

    if (ktiles > 0) issue(0, 0);
    for (int64_t kt = 0; kt < ktiles; ++kt) {
        const int stage = (int)(kt & 1);
        if (kt + 1 < ktiles) {
            issue(kt + 1, stage ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const uint32_t *As = smem + stage * stage_words;
        const uint32_t *Bs = As + a_stage_words;
#pragma unroll 2
        for (int kw = 0; kw < KT; ++kw) {
            for (int i = 0; i < ka; ++i) {
                uint32_t af[TM];
                const uint32_t *ap = As + (i * KT + kw) * (BM + PADW) + ty * TM;
#pragma unroll
                for (int r = 0; r < TM; r += 4) {
                    const uint4 v = *reinterpret_cast<const uint4 *>(ap + r);
                    af[r] = v.x; af[r + 1] = v.y; af[r + 2] = v.z; af[r + 3] = v.w;
                }
                if (MODE == M_AND_SA) {
#pragma unroll
                    for (int r = 0; r < TM; ++r) sa[r] += __popc(af[r]) << i;
                }
                for (int j = 0; j < kb; ++j) {
                    uint32_t bf[TN];
                    const uint32_t *bp = Bs + (j * KT + kw) * (BN + PADW) + tx * 4;
#pragma unroll
                    for (int q = 0; q < G; ++q) {
                        const uint4 v = *reinterpret_cast<const uint4 *>(bp + q * GSTRIDE);
                        bf[4 * q] = v.x; bf[4 * q + 1] = v.y; bf[4 * q + 2] = v.z; bf[4 * q + 3] = v.w;
                    }
                    if (MODE == M_AND_SB) {
                        if (i == 0) {
#pragma unroll
                            for (int c = 0; c < TN; ++c) sb[c] += __popc(bf[c]) << j;
                        }
                    }
                    const int sh = i + j;
#pragma unroll
                    for (int r = 0; r < TM; ++r)
#pragma unroll
                        for (int c = 0; c < TN; ++c) {
                            const uint32_t x = (MODE == M_XOR) ? (af[r] ^ bf[c]) : (af[r] & bf[c]);
                            if (SINGLE) acc[r][c] += __popc(x);
                            else acc[r][c] += __popc(x) << sh;
                        }
                }
            }
        }
        __syncthreads();
    }

    // ---- epilogue ----------------------------------------------------------
    const bool want_bits = (g.out_bits != nullptr);
    const bool want_int = (g.out != nullptr);
    const int lane = tid & 31;
#pragma unroll
    for (int r = 0; r < TM; ++r) {
        const int64_t m = m0 + ty * TM + r;
        const bool mrow = m < g.M;
#pragma unroll
        for (int q = 0; q < G; ++q) {
            const int64_t nb = n0 + q * GSTRIDE + tx * 4;
            int32_t v[4];
            uint32_t nib = 0;
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                const int c = 4 * q + c4;
                int32_t val;
                if (MODE == M_XOR) val = P.kll - 2 * acc[r][c];
                else if (MODE == M_AND_SA) val = 2 * acc[r][c] - P.lb * sa[r];
                else if (MODE == M_AND_SB) val = 2 * acc[r][c] - P.la * sb[c];
                else val = acc[r][c];
                v[c4] = val;
                if (want_bits && mrow && (nb + c4) < g.N) {
                    uint32_t b = val >= __ldg(g.thr + nb + c4);
                    if (g.flip) b ^= (uint32_t)(__ldg(g.flip + nb + c4) != 0);
                    nib |= b << c4;
                }
            }
            if (want_int && mrow) {
                if (g.epilogue == EPI_NCHW) {
                    const int64_t img = m / g.hw;
                    const int64_t pix = m - img * g.hw;
#pragma unroll
                    for (int c4 = 0; c4 < 4; ++c4)
                        if (nb + c4 < g.N) g.out[(img * g.N + nb + c4) * g.hw + pix] = v[c4];
                } else {
                    int32_t *dst = g.out + m * g.ldo + nb;
                    if (nb + 4 <= g.N && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
                        *reinterpret_cast<int4 *>(dst) = make_int4(v[0], v[1], v[2], v[3]);
                    } else {
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4)
                            if (nb + c4 < g.N) dst[c4] = v[c4];
                    }
                }
            }
            if (want_bits) {   // uniform branch: every lane takes part in the shuffles
                uint32_t w = nib << (4 * (lane & 7));
                w |= __shfl_xor_sync(0xffffffffu, w, 1);
                w |= __shfl_xor_sync(0xffffffffu, w, 2);
                w |= __shfl_xor_sync(0xffffffffu, w, 4);
                if ((lane & 7) == 0 && mrow && nb < g.N) g.out_bits[m * g.ld_bits + (nb >> 5)] = w;
            }
        }
    }
}

// Few output units (a classifier head: N <= 16), 1-bit x 1-bit: the work is one pass over the packed
// activations, so the kernel is a streaming one.  B's rows sit in shared memory; a warp owns FOUR rows
// of A at a time, eight lanes per row, each lane xor/popc-ing every eighth 128-bit chunk of its row
// against all N rows of B; the N partial counts are then summed over the eight lanes (three shuffle
// steps instead of five over a whole warp).
constexpr int SKINNY_N = 16;
__global__ void __launch_bounds__(256) gemm_popc_skinny_kernel(const uint32_t *__restrict__ a, int64_t lda,
                                                               const uint32_t *__restrict__ b, int64_t ldb, int64_t M,
                                                               int N, int64_t kwords, int32_t K, int32_t *__restrict__ out,
                                                               int64_t ldo)
{
    extern __shared__ __align__(16) uint32_t bs[];               // [N][kw4], kw4 = kwords rounded up to 4, zero padded
    const int kw4 = (int)((kwords + 3) & ~(int64_t)3);
    griddep_launch_dependents();
    griddep_wait();                                              // (the weights could be read before this; the activations not)
    for (int e = threadIdx.x; e < N * kw4; e += blockDim.x) {
        const int n = e / kw4, k = e - n * kw4;
        bs[e] = k < kwords ? __ldg(b + (int64_t)n * ldb + k) : 0u;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int sub = lane >> 3;                                   // which of the warp's four rows
    const int part = lane & 7;                                   // which eighth of the row's chunks
    const int64_t warp0 = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const bool vec = ((lda & 3) == 0) && ((reinterpret_cast<uintptr_t>(a) & 15) == 0);
    for (int64_t m0 = warp0 * 4; m0 < M; m0 += nwarps * 4) {
        const int64_t m = m0 + sub;
        const bool live = m < M;
        int32_t acc[SKINNY_N];
#pragma unroll
        for (int n = 0; n < SKINNY_N; ++n) acc[n] = 0;
        const uint32_t *arow = a + (live ? m : m0) * lda;
        // four 16-byte pieces of the row per lane are loaded before any of them is used: the kernel is a stream over A,
        // and one load in flight per lane leaves it waiting out a memory latency per piece
        for (int k0 = part * 4; k0 < kwords; k0 += 128) {
            uint4 av[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int k = k0 + 32 * u;
                if (vec && k + 4 <= kwords) {
                    av[u] = __ldcs(reinterpret_cast<const uint4 *>(arow + k));
                } else {
                    av[u].x = k < kwords ? arow[k] : 0u;
                    av[u].y = k + 1 < kwords ? arow[k + 1] : 0u;
                    av[u].z = k + 2 < kwords ? arow[k + 2] : 0u;
                    av[u].w = k + 3 < kwords ? arow[k + 3] : 0u;
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int k = k0 + 32 * u;
                if (k < kwords) {
#pragma unroll
                    for (int n = 0; n < SKINNY_N; ++n) {
                        if (n < N) {
                            const uint4 bv = *reinterpret_cast<const uint4 *>(bs + n * kw4 + k);
                            acc[n] += __popc(av[u].x ^ bv.x) + __popc(av[u].y ^ bv.y) + __popc(av[u].z ^ bv.z) + __popc(av[u].w ^ bv.w);
                        }
                    }
                }
            }
        }
        int32_t lo = 0, hi = 0;                                  // lane `part` keeps units part and part + 8 of its row
#pragma unroll
        for (int n = 0; n < SKINNY_N; ++n) {
            if (n < N) {
                int32_t v = acc[n];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                v += __shfl_xor_sync(0xffffffffu, v, 4);
                if ((n & 7) == part) { if (n < 8) lo = v; else hi = v; }
            }
        }
        if (live) {
            if (part < N) out[m * ldo + part] = K - 2 * lo;
            if (part + 8 < N) out[m * ldo + part + 8] = K - 2 * hi;
        }
    }
}

int launch_skinny(const PopcParams &P, cudaStream_t st)
{
    const GemmArgs &g = P.g;
    const int64_t kw4 = (P.kwords + 3) & ~(int64_t)3;
    const size_t smem = sizeof(uint32_t) * (size_t)g.N * (size_t)kw4;
    auto kern = gemm_popc_skinny_kernel;
    if (smem > 48 * 1024) QNN_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    // a warp takes four rows per pass, a block 32
    const int64_t need = ceil_div(g.M, 32);
    const int64_t cap = (int64_t)sm_count() * 4;
    const int blocks = (int)(need < cap ? need : cap);
    profile_before(st);
    QNN_CUDA(launch_pdl(kern, dim3(blocks), dim3(256), smem, st, g.a, g.lda, g.b, g.ldb, g.M, (int)g.N, P.kwords, P.kll, g.out, g.ldo));
    profile_after(st);
    return check_launch("popc gemm (few units)");
}

template <int BM, int BN, int TM, int TN, int MODE, bool SINGLE>
int launch_cfg(const PopcParams &P, cudaStream_t st)
{
    const GemmArgs &g = P.g;
    const int ka = SINGLE ? 1 : g.ka, kb = SINGLE ? 1 : g.kb;
    const size_t smem = 2u * sizeof(uint32_t) * (size_t)(ka * KT * (BM + PADW) + kb * KT * (BN + PADW));
    auto kern = gemm_popc_kernel<BM, BN, TM, TN, MODE, SINGLE>;
    if (smem > 48 * 1024) {
        QNN_REQUIRE(smem <= 227 * 1024, QNN_ERR_UNSUPPORTED, "popc gemm: %d x %d planes need %zu bytes of shared memory",
                    ka, kb, smem);
        QNN_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    const int64_t gx = ceil_div(g.N, BN), gy = ceil_div(g.M, BM);
    QNN_REQUIRE(gy <= 65535, QNN_ERR_UNSUPPORTED, "popc gemm: M too large for the launch grid");
    dim3 grid((unsigned)gx, (unsigned)gy);
    profile_before(st);
    kern<<<grid, THREADS, smem, st>>>(P);
    profile_after(st);
    return check_launch("popc gemm");
}

template <int MODE, bool SINGLE>
int launch_mode(const PopcParams &P, cudaStream_t st)
{
    const GemmArgs &g = P.g;
    const int64_t big_tiles = ceil_div(g.M, 128) * ceil_div(g.N, 128);
    // multi-plane A tiles are large in shared memory; keep those on the small tile too when planes are many
    const bool small = big_tiles < sm_count() || (!SINGLE && (g.ka + g.kb) > 9);
    if (small) return launch_cfg<64, 64, 4, 4, MODE, SINGLE>(P, st);
    return launch_cfg<128, 128, 8, 8, MODE, SINGLE>(P, st);
}

}  // namespace

int launch_gemm_popc(const GemmArgs &g, cudaStream_t st)
{
    if (g.M == 0 || g.N == 0) return QNN_OK;
    PopcParams P;
    P.g = g;
    P.kwords = g.kwords > 0 ? g.kwords : ceil_div(g.K, 32);
    P.la = (1 << g.ka) - 1;
    P.lb = (1 << g.kb) - 1;
    P.kll = (int32_t)(g.K * P.la * P.lb);
    const bool a_pm = g.a_mode == QNN_MODE_PM1, b_pm = g.b_mode == QNN_MODE_PM1;
    if (a_pm && b_pm) {
        if (g.ka == 1 && g.kb == 1) {
            const bool skinny = g.N <= SKINNY_N && g.M >= 64 && g.epilogue == EPI_ROWMAJOR && g.out != nullptr &&
                                g.out_bits == nullptr && g.kwords == 0 &&
                                sizeof(uint32_t) * (size_t)g.N * (size_t)(P.kwords + 3) <= 160 * 1024;
            if (skinny) return launch_skinny(P, st);
            return launch_mode<M_XOR, true>(P, st);
        }
        return launch_mode<M_XOR, false>(P, st);
    }
    if (!a_pm && b_pm) return launch_mode<M_AND_SA, false>(P, st);
    if (a_pm && !b_pm) return launch_mode<M_AND_SB, false>(P, st);
    return launch_mode<M_AND, false>(P, st);
}

}  // namespace qnn
