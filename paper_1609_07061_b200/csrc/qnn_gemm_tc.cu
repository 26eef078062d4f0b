// Tensor-core matrix product: the packed operands are expanded to their int8
// VALUES (+-1, unsigned codes or signed-symmetric codes; pad positions become
// 0) in the caller's workspace, then one persistent, warp-specialised kernel
// multiplies them on the 5th-generation tensor cores:
//   TMA (128-byte swizzle) -> shared-memory ring -> tcgen05.mma kind::i8 with
//   the int32 accumulator in tensor memory (two accumulator stages) ->
//   tcgen05.ld epilogue (int32 rows, NCHW scatter or threshold -> packed bits).
// One int8 multiply-accumulate carries one product of the paper's sum, so a
// k-bit x k-bit product costs ONE pass here instead of ka*kb plane passes.
//
// Every device-side wait is bounded: when a wait runs out the kernel records a
// code in a device status word, raises a block-wide abort flag, lets copies in
// flight land, frees its tensor memory and returns.
#include <cuda.h>
#include "qnn_internal.cuh"

namespace qnn {
namespace {

constexpr int BM = 128;              // rows of A per tile (UMMA M)
constexpr int BK = 128;              // int8 elements of K per pipeline stage = one 128-byte swizzle row
constexpr int UMMA_K = 32;           // K per tcgen05.mma of kind::i8
constexpr int TC_THREADS = 192;      // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2..5: epilogue
constexpr uint32_t WAIT_LIMIT = 1u << 22;

__device__ int g_tc_status = 0;      // 0 = fine; otherwise the code of the first wait that ran out

struct TcParams {
    int64_t M, N;
    int32_t num_kb;                  // K blocks of BK
    int32_t tiles_m, tiles_n;
    int epilogue;
    int32_t *out; int64_t ldo; int64_t hw;
    const int32_t *thr; const uint8_t *flip; uint32_t *out_bits; int64_t ld_bits;
    uint32_t idesc;
};

// ---- PTX wrappers -----------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the block is aborting (this wait ran out, or another one did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int code)
{
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 128) __nanosleep(64);
        if ((it & 63) == 63 && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(&g_tc_status, 0, code);
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled
// (the layout a TMA box of 128 bytes x rows produces): 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t saddr)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3ffffu) >> 4);          // start address, 16-byte units
    d |= (uint64_t)1 << 16;                            // leading-dimension offset (unused with swizzle) = 1
    d |= (uint64_t)(1024 >> 4) << 32;                  // stride between 8-row groups
    d |= (uint64_t)1 << 46;                            // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                            // 128-byte swizzle
    return d;
}

template <int BN>
struct TcSmem {
    static constexpr int STAGES = (BN == 256) ? 4 : (BN == 128 ? 6 : 8);
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_BYTES = BN * BK;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int TMEM_COLS = (2 * BN < 32) ? 32 : 2 * BN;     // two accumulator stages
    static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
    static constexpr int TOTAL = BAR_OFFSET + 256 + 1024;              // barriers + slack for 1024-byte alignment
};

template <int BN>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const TcParams p)
{
    using S = TcSmem<BN>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;                      // swizzled tiles need 1024-byte alignment
    uint8_t *gen = smem_raw + (base - raw);
    uint64_t *bars = reinterpret_cast<uint64_t *>(gen + S::BAR_OFFSET);
    const uint32_t bar0 = base + S::BAR_OFFSET;
    auto full_bar = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (uint32_t)(S::STAGES + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (uint32_t)(2 * S::STAGES + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (uint32_t)(2 * S::STAGES + 2 + a); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * S::STAGES + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 128); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), S::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int64_t num_tiles = (int64_t)p.tiles_m * p.tiles_n;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
                const int32_t tm = (int32_t)(t % p.tiles_m), tn = (int32_t)(t / p.tiles_m);
                for (int32_t kb = 0; kb < p.num_kb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 1)) { ok = false; break; }
                    mbar_expect_tx(full_bar(stage), (uint32_t)S::STAGE_BYTES);
                    const uint32_t sa = base + (uint32_t)stage * S::STAGE_BYTES;
                    tma_load_2d(sa, &tmap_a, kb * BK, tm * BM, full_bar(stage));
                    tma_load_2d(sa + S::A_BYTES, &tmap_b, kb * BK, tn * BN, full_bar(stage));
                    if (++stage == S::STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            uint32_t iter = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++iter) {
                const uint32_t as = iter & 1u, aphase = (iter >> 1) & 1u;
                if (!mbar_wait(tempty_bar(as), aphase ^ 1u, abort_flag, 2)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + as * (uint32_t)BN;
                for (int32_t kb = 0; kb < p.num_kb; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, 3)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = base + (uint32_t)stage * S::STAGE_BYTES;
                    const uint64_t adesc = make_kmajor_sw128_desc(sa);
                    const uint64_t bdesc = make_kmajor_sw128_desc(sa + S::A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        // advancing K inside the swizzle row: +32 bytes = +2 in the 16-byte address field
                        umma_i8(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), p.idesc,
                                (uint32_t)((kb | k) != 0));
                    }
                    umma_commit(empty_bar(stage));               // frees the smem slot once these MMAs retire
                    if (++stage == S::STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(tfull_bar(as));              // accumulator complete
            }
        }
    } else {
        const int q = warp & 3;                                  // TMEM lane quarter this warp may read
        uint32_t iter = 0;
        bool ok = true;
        for (int64_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++iter) {
            const int32_t tm = (int32_t)(t % p.tiles_m), tn = (int32_t)(t / p.tiles_m);
            const uint32_t as = iter & 1u, aphase = (iter >> 1) & 1u;
            // the tensor-memory loads below are warp-collective: leave the loop only as a whole warp
            if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(as), aphase, abort_flag, 4))) { ok = false; break; }
            tc_fence_after();
            const int64_t m = (int64_t)tm * BM + q * 32 + lane;
            const bool mrow = m < p.M;
            int64_t img = 0, pix = 0;
            if (p.epilogue == EPI_NCHW && mrow) { img = m / p.hw; pix = m - img * p.hw; }
            uint32_t words[BN / 32];
#pragma unroll
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + as * (uint32_t)BN + (uint32_t)(c * 32), v);
                const int64_t n0 = (int64_t)tn * BN + c * 32;
                if (p.out != nullptr && mrow && n0 < p.N) {
                    if (p.epilogue == EPI_NCHW) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + j < p.N) p.out[(img * p.N + n0 + j) * p.hw + pix] = (int32_t)v[j];
                    } else {
                        int32_t *dst = p.out + m * p.ldo + n0;
                        if (n0 + 32 <= p.N && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<int4 *>(dst + j) = make_int4((int)v[j], (int)v[j + 1], (int)v[j + 2], (int)v[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (n0 + j < p.N) dst[j] = (int32_t)v[j];
                        }
                    }
                }
                uint32_t w = 0;
                if (p.out_bits != nullptr && n0 < p.N) {
                    // lane j fetches the threshold (and flip) of column n0 + j once; the row loop reads them by shuffle
                    const bool ncol = (n0 + lane) < p.N;
                    const int32_t tl = ncol ? __ldg(p.thr + n0 + lane) : 0;
                    const uint32_t fl = (ncol && p.flip) ? (uint32_t)(__ldg(p.flip + n0 + lane) != 0) : 0u;
                    const uint32_t fmask = __ballot_sync(0xffffffffu, fl != 0);
                    const uint32_t nmask = __ballot_sync(0xffffffffu, ncol);
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int32_t tj = __shfl_sync(0xffffffffu, tl, j);
                        w |= (uint32_t)((int32_t)v[j] >= tj) << j;
                    }
                    w = (w ^ fmask) & nmask;
                }
                words[c] = w;
            }
            // all TMEM reads of this accumulator stage are done: hand it back to the MMA warp
            tc_fence_before();
            mbar_arrive(tempty_bar(as));
            if (p.out_bits != nullptr && mrow) {
                uint32_t *dst = p.out_bits + m * p.ld_bits + (((int64_t)tn * BN) >> 5);
#pragma unroll
                for (int c = 0; c < BN / 32; ++c)
                    if ((int64_t)tn * BN + c * 32 < p.N) dst[c] = words[c];
            }
        }
    }

    // ---- teardown ------------------------------------------------------------
    __syncwarp();
    if (*abort_flag) {
        // give copies and MMAs still in flight time to land before shared and tensor memory are released
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, S::TMEM_COLS);
}

// ---- expansion of packed planes to int8 values ------------------------------

// One thread produces 16 consecutive bytes of a row.  `period`/`tail` describe where pad bits sit:
// word (w mod period) == period-1 has only `tail` valid bits; every pad position expands to 0.
__global__ void __launch_bounds__(256) expand_i8_kernel(const uint32_t *__restrict__ planes, int nplanes, int pm1,
                                                        int64_t ld, int64_t plane_stride, int64_t rows, int64_t kwords,
                                                        int64_t period, int tail, int64_t kp, uint8_t *__restrict__ out)
{
    const int64_t chunks = kp >> 4;
    const int64_t total = rows * chunks;
    const uint32_t lcode = (1u << nplanes) - 1u;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = e / chunks;
        const int64_t ch = e - r * chunks;
        const int64_t widx = ch >> 1;
        const int half = (int)(ch & 1);
        uint32_t o[4] = {0u, 0u, 0u, 0u};
        if (widx < kwords) {
            const int valid = ((widx % period) == period - 1) ? tail : 32;
            const uint32_t vword = (valid >= 32) ? 0xffffffffu : ((1u << valid) - 1u);
            const uint32_t vm = (vword >> (16 * half)) & 0xffffu;
            uint32_t acc[4] = {0u, 0u, 0u, 0u};
            for (int i = 0; i < nplanes; ++i) {
                const uint32_t w = __ldg(planes + i * plane_stride + r * ld + widx);
                const uint32_t h = (w >> (16 * half)) & 0xffffu;
#pragma unroll
                for (int nb = 0; nb < 4; ++nb) {
                    const uint32_t nib = (h >> (4 * nb)) & 0xfu;
                    acc[nb] += ((nib * 0x00204081u) & 0x01010101u) << i;       // bit j of the nibble -> byte j
                }
            }
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) {
                uint32_t v = acc[nb];
                if (pm1) v = __vsub4(v << 1, lcode * 0x01010101u);              // 2q - (2^k - 1) per byte
                const uint32_t mnib = (vm >> (4 * nb)) & 0xfu;
                const uint32_t mask = ((mnib * 0x00204081u) & 0x01010101u) * 0xffu;
                o[nb] = v & mask;
            }
        }
        *reinterpret_cast<uint4 *>(out + r * kp + ch * 16) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

int make_map(CUtensorMap *map, const uint8_t *base, int64_t rows, int64_t kp, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    QNN_REQUIRE(fn != nullptr, QNN_ERR_CUDA, "tc gemm: cuTensorMapEncodeTiled is not available from this driver");
    cuuint64_t dims[2] = {(cuuint64_t)kp, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)kp};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    QNN_REQUIRE(r == CUDA_SUCCESS, QNN_ERR_CUDA, "tc gemm: cuTensorMapEncodeTiled failed with code %d", (int)r);
    return QNN_OK;
}

template <int BN>
int launch_tc_cfg(const CUtensorMap &ma, const CUtensorMap &mb, TcParams p, cudaStream_t st)
{
    using S = TcSmem<BN>;
    auto kern = gemm_i8_kernel<BN>;
    QNN_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL));
    p.tiles_n = (int32_t)ceil_div(p.N, BN);
    p.idesc |= (uint32_t)(BN >> 3) << 17;
    const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n;
    const int grid = (int)(tiles < sm_count() ? tiles : sm_count());
    profile_before(st);
    kern<<<grid, TC_THREADS, S::TOTAL, st>>>(ma, mb, p);
    profile_after(st);
    return check_launch("tc gemm");
}

inline int64_t kp_of(int64_t kwords) { return (int64_t)round_up((size_t)kwords * 32, BK); }

}  // namespace

bool gemm_tc_supported(const GemmArgs &g)
{
    // signed-symmetric codes of 8 planes reach +-255 and do not fit int8
    if (g.a_mode == QNN_MODE_PM1 && g.ka > 7) return false;
    if (g.b_mode == QNN_MODE_PM1 && g.kb > 7) return false;
    if (g.M > (int64_t)1 << 30 || g.N > (int64_t)1 << 30) return false;
    return true;
}

size_t gemm_tc_workspace_bytes(int64_t M, int64_t N, int64_t K, int, int)
{
    const int64_t kp = kp_of(ceil_div(K, 32));
    return round_up((size_t)M * (size_t)kp, 256) + round_up((size_t)N * (size_t)kp, 256);
}

int launch_gemm_tc(const GemmArgs &g, void *ws, size_t ws_bytes, cudaStream_t st)
{
    QNN_REQUIRE(gemm_tc_supported(g), QNN_ERR_UNSUPPORTED,
                "tc gemm: signed-symmetric operands of 8 planes do not fit int8; use QNN_ALGO_POPC");
    const int64_t kwords = g.kwords > 0 ? g.kwords : ceil_div(g.K, 32);
    QNN_REQUIRE(kwords > 0, QNN_ERR_UNSUPPORTED, "tc gemm: K = 0 is handled by QNN_ALGO_POPC");
    const int64_t kp = kp_of(kwords);
    const size_t a_bytes = round_up((size_t)g.M * (size_t)kp, 256);
    const size_t need = a_bytes + round_up((size_t)g.N * (size_t)kp, 256);
    QNN_REQUIRE(ws != nullptr && aligned(ws, 256) && ws_bytes >= need, QNN_ERR_WORKSPACE,
                "tc gemm: workspace of at least %zu bytes (256-byte aligned) required", need);
    QNN_REQUIRE(kp / BK < ((int64_t)1 << 31), QNN_ERR_UNSUPPORTED, "tc gemm: K too large");
    uint8_t *a8 = static_cast<uint8_t *>(ws);
    uint8_t *b8 = a8 + a_bytes;

    // where the pad bits are: a plain matrix pads only its last word; conv rows pad the last word of every tap
    int64_t period = kwords;
    int tail = (int)(g.K - 32 * (kwords - 1));
    if (g.pad_period > 0) { period = g.pad_period; tail = g.pad_tail; }
    QNN_REQUIRE(tail >= 1 && tail <= 32, QNN_ERR_INVALID_ARG, "tc gemm: inconsistent K / kwords");

    auto expand = [&](const uint32_t *src, int planes, int mode, int64_t ld, int64_t stride, int64_t rows, uint8_t *dst) {
        const int64_t total = rows * (kp >> 4);
        const int64_t need_blocks = ceil_div(total, 256);
        const int64_t cap = (int64_t)sm_count() * 16;
        const int blocks = (int)(need_blocks < cap ? need_blocks : cap);
        expand_i8_kernel<<<blocks, 256, 0, st>>>(src, planes, mode == QNN_MODE_PM1, ld, stride, rows, kwords, period, tail,
                                                 kp, dst);
        return check_launch("tc gemm expand");
    };
    if (int rc = expand(g.a, g.ka, g.a_mode, g.lda, g.a_plane_stride, g.M, a8)) return rc;
    if (int rc = expand(g.b, g.kb, g.b_mode, g.ldb, g.b_plane_stride, g.N, b8)) return rc;

    TcParams p{};
    p.M = g.M; p.N = g.N; p.num_kb = (int32_t)(kp / BK);
    p.tiles_m = (int32_t)ceil_div(g.M, BM);
    p.epilogue = g.epilogue; p.out = g.out; p.ldo = g.ldo; p.hw = g.hw > 0 ? g.hw : 1;
    p.thr = g.thr; p.flip = g.flip; p.out_bits = g.out_bits; p.ld_bits = g.ld_bits;
    // instruction descriptor: int32 accumulator, A/B int8 signed (PM1) or unsigned (U01), both K-major, M = 128
    p.idesc = (2u << 4) | ((g.a_mode == QNN_MODE_PM1 ? 1u : 0u) << 7) | ((g.b_mode == QNN_MODE_PM1 ? 1u : 0u) << 10) |
              ((uint32_t)(BM >> 4) << 24);

    // widest tile that still gives every SM work
    const int64_t tm = p.tiles_m;
    int bn = 256;
    if (tm * ceil_div(g.N, 256) < sm_count()) bn = 128;
    if (bn == 128 && tm * ceil_div(g.N, 128) < sm_count()) bn = 64;
    CUtensorMap ma, mb;
    if (int rc = make_map(&ma, a8, g.M, kp, BM)) return rc;
    if (int rc = make_map(&mb, b8, g.N, kp, bn)) return rc;
    if (bn == 256) return launch_tc_cfg<256>(ma, mb, p, st);
    if (bn == 128) return launch_tc_cfg<128>(ma, mb, p, st);
    return launch_tc_cfg<64>(ma, mb, p, st);
}

}  // namespace qnn

extern "C" int qnn_device_status(void *stream)
{
    using namespace qnn;
    QNN_CUDA(cudaStreamSynchronize(as_stream(stream)));
    int code = 0;
    QNN_CUDA(cudaMemcpyFromSymbol(&code, g_tc_status, sizeof(int)));
    if (code != 0) {
        const int zero = 0;
        QNN_CUDA(cudaMemcpyToSymbol(g_tc_status, &zero, sizeof(int)));
        return fail(QNN_ERR_TIMEOUT, "a bounded device-side wait ran out (wait site %d)", code);
    }
    return QNN_OK;
}
