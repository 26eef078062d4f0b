// Matrix product for SMALL batches straight from packed bit-planes (Eq. 11's operands as they cross the ABI), on the
// tensor cores, in one launch and without a workspace:
//     TMA brings PACKED tiles (32 elements per word) into shared memory -- 2048 (or 1024) elements of K per row at a time;
//     converter warps expand them to one e2m1 value per element directly into the 128-byte-swizzled operand tiles
//     that tcgen05.mma reads (the expanded operands never exist in global memory);
//     one thread issues the block-scaled e2m1 products (unit scales, fp32 accumulation in tensor memory: exact
//     integers below 2^24);  four warps turn the accumulators into int32 rows or thresholded bits.
// With few rows in A there is too little work per weight for the rewriting of the operands (two more launches and
// 4x the packed bytes through HBM) to pay off; for large batches the prepared-operand kernel remains the faster one.
//
//   warp 0        TMA: packed A and B tiles
//   warp 1        tcgen05.mma issue, tensor-memory owner
//   warps 2..5    epilogue
//   warps 6..21   converters
//
// Operands: up to 2 planes each, {0,1} codes or +-1 values (the value sets e2m1 holds).  Every device-side wait is bounded.
#include <atomic>
#include "qnn_internal.cuh"
#include "qnn_tc_ptx.cuh"

namespace qnn {
namespace {

constexpr int SM_BN = 32;                       // output columns per CTA
constexpr int SM_KB = 256;                      // k per operand stage (128 bytes of e2m1)
constexpr int SM_SB_WORDS = 64;                 // packed words of K per row in one packed tile (2048 elements); 32 when four planes have to fit
constexpr int SM_CONV_WARPS = 16;               // (the kernel is bound by the converters' instruction stream: 16 warps hide more latency than 8)
constexpr int SM_CONV_THREADS = 32 * SM_CONV_WARPS;
constexpr int SM_A_ITEMS = BM * 8 / SM_CONV_THREADS;   // packed A words a converter thread expands per operand stage: 2
constexpr int SM_THREADS = 32 * (6 + SM_CONV_WARPS);
constexpr int SM_A_BYTES = BM * BKB;            // 16 KB
constexpr int SM_B_BYTES = SM_BN * BKB;         // 4 KB
constexpr int SM_STAGE_BYTES = SM_A_BYTES + SM_B_BYTES;
constexpr int SM_STAGES = 4;
constexpr int SM_PACKED_BUFS = 2;

struct SmParams {
    int64_t M, N, K;
    int32_t num_sb;                              // packed tiles along K
    int32_t sbw;                                 // packed words of K per row in one packed tile
    int32_t ka, kb, a_pm1, b_pm1;
    int32_t pa_bytes, pb_bytes;                  // bytes of one packed A / B tile (all planes)
    int32_t *out; int64_t ldo;
    const int32_t *thr; const uint8_t *flip; uint32_t *out_bits; int64_t ld_bits;
    uint32_t idesc;
};

// 32 elements of up to two planes as 32 e2m1 values (element 2i in the low nibble of byte i); elements outside `valid` -> 0
__device__ __forceinline__ uint4 planes_to_fp4(uint32_t p0, uint32_t p1, int nplanes, int pm1, uint32_t valid)
{
    uint32_t o[4];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        const uint32_t s0 = spread_bits_to_nibbles((p0 >> (8 * b)) & 0xffu);
        uint32_t code;
        if (pm1) {
            if (nplanes == 1) {
                code = 0xAAAAAAAAu ^ (s0 << 3);                            // bit 1 -> +1 (0x2), bit 0 -> -1 (0xA)
            } else {
                // value 2*q - 3 with q = s0 + 2*s1: q 0 -> -3, 1 -> -1, 2 -> +1, 3 -> +3
                const uint32_t s1 = spread_bits_to_nibbles((p1 >> (8 * b)) & 0xffu);
                const uint32_t neg = (s1 ^ 0x11111111u) << 3;
                const uint32_t three = ~(s0 ^ s1) & 0x11111111u;
                code = neg | (three * 0x5u) | ((three ^ 0x11111111u) << 1);
            }
        } else {
            // unsigned code q = s0 + 2*s1: 0 -> 0, 1 -> 0b010, 2 -> 0b100, 3 -> 0b101
            const uint32_t s1 = nplanes > 1 ? spread_bits_to_nibbles((p1 >> (8 * b)) & 0xffu) : 0u;
            code = (s1 << 2) | ((s0 & ~s1) << 1) | (s0 & s1);
        }
        o[b] = code & (spread_bits_to_nibbles((valid >> (8 * b)) & 0xffu) * 0xfu);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// 32 sign bits as 32 e2m1 values, no pad elements: +1 -> 0x2, -1 -> 0xA
__device__ __forceinline__ uint4 signs_to_fp4_full(uint32_t w)
{
    return make_uint4(0xAAAAAAAAu ^ (spread_bits_to_nibbles(w & 0xffu) << 3), 0xAAAAAAAAu ^ (spread_bits_to_nibbles((w >> 8) & 0xffu) << 3),
                      0xAAAAAAAAu ^ (spread_bits_to_nibbles((w >> 16) & 0xffu) << 3), 0xAAAAAAAAu ^ (spread_bits_to_nibbles(w >> 24) << 3));
}

__global__ void __launch_bounds__(SM_THREADS, 1)
gemm_smallm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const SmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - raw);
    // layout: operand stages | packed tiles (A planes, then B planes, per buffer) | barriers
    const int packed_bytes = p.pa_bytes + p.pb_bytes;
    const int packed_off = SM_STAGES * SM_STAGE_BYTES;
    const int bar_off = packed_off + SM_PACKED_BUFS * packed_bytes;
    const uint32_t bar0 = base + (uint32_t)bar_off;
    uint64_t *bars = reinterpret_cast<uint64_t *>(gen + bar_off);
    auto full_bar = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (uint32_t)(SM_STAGES + s); };
    const uint32_t tfull_bar = bar0 + 8u * (uint32_t)(2 * SM_STAGES);
    auto pfull_bar = [&](int b) { return bar0 + 8u * (uint32_t)(2 * SM_STAGES + 1 + b); };
    auto pempty_bar = [&](int b) { return bar0 + 8u * (uint32_t)(2 * SM_STAGES + 1 + SM_PACKED_BUFS + b); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * SM_STAGES + 1 + 2 * SM_PACKED_BUFS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int64_t n0 = (int64_t)blockIdx.x * SM_BN;
    const int32_t m0 = (int32_t)blockIdx.y * BM;
    const int32_t num_kb = (int32_t)((p.K + SM_KB - 1) / SM_KB);
    griddep_launch_dependents();

    if (threadIdx.x == 0) {
        for (int s = 0; s < SM_STAGES; ++s) { mbar_init(full_bar(s), SM_CONV_WARPS); mbar_init(empty_bar(s), 1); }
        mbar_init(tfull_bar, 1);
        for (int b = 0; b < SM_PACKED_BUFS; ++b) { mbar_init(pfull_bar(b), 1); mbar_init(pempty_bar(b), SM_CONV_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // The four K steps of an operand stage go to FOUR accumulators (each sums every fourth step) which the epilogue adds:
    // with one accumulator every product would wait for the one before it, and at 32 columns a product is far shorter
    // than the pipe's latency -- the chain of dependent products, not the work, would set the pace.
    constexpr int NACC = 4;
    constexpr uint32_t SCALE_COL = NACC * SM_BN;   // 128 accumulator columns, then 32 columns of unit scales
    constexpr uint32_t TMEM_COLS = 256;
    if (warp == 1) tmem_alloc<1>(smem_u32(tmem_slot), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (warp >= 2 && warp < 6) {
        const int q = warp & 3;
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_st8(tmem_base + ((uint32_t)(q * 32) << 16) + SCALE_COL + (uint32_t)(8 * c), 0x7f7f7f7fu);
        tmem_st_wait();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    griddep_wait();                                  // both operands may come from the kernel before this one

    if (warp == 0) {
        if (lane == 0) {
            // packed tiles: per plane one box of 64 words x 128 rows (A) / 32 rows (B), dense rows of 256 bytes
            int buf = 0; uint32_t phase = 0;
            for (int32_t sb = 0; sb < p.num_sb; ++sb) {
                if (!mbar_wait(pempty_bar(buf), phase ^ 1u, abort_flag, 21)) break;
                const uint32_t dst = base + (uint32_t)(packed_off + buf * packed_bytes);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(pfull_bar(buf)), "r"((uint32_t)packed_bytes) : "memory");
                for (int pl = 0; pl < p.ka; ++pl)
                    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                                 ::"r"(dst + (uint32_t)(pl * BM * p.sbw * 4)), "l"(&tmap_a), "r"(sb * p.sbw), "r"(m0), "r"(pl),
                                   "r"(pfull_bar(buf)) : "memory");
                for (int pl = 0; pl < p.kb; ++pl)
                    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                                 ::"r"(dst + (uint32_t)(p.pa_bytes + pl * SM_BN * p.sbw * 4)), "l"(&tmap_b), "r"(sb * p.sbw),
                                   "r"((int32_t)n0), "r"(pl), "r"(pfull_bar(buf)) : "memory");
                if (++buf == SM_PACKED_BUFS) { buf = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            const uint32_t sf = tmem_base + SCALE_COL;
            for (int32_t kb = 0; kb < num_kb && ok; ++kb) {
                if (!mbar_wait(full_bar(stage), phase, abort_flag, 22)) { ok = false; break; }
                tc_fence_after();
                const uint32_t sa = base + (uint32_t)(stage * SM_STAGE_BYTES);
                const uint64_t da = make_kmajor_desc<BKB>(sa), db = make_kmajor_desc<BKB>(sa + SM_A_BYTES);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint64_t a = da + (uint64_t)(2 * ks), b = db + (uint64_t)(2 * ks);
                    const uint32_t acc = kb != 0;
                    asm volatile("{\n.reg .pred P;\nsetp.ne.b32 P, %4, 0;\n"
                                 "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%5], P;\n}\n"
                                 ::"r"(tmem_base + (uint32_t)(ks * SM_BN)), "l"(a), "l"(b), "r"(p.idesc), "r"(acc), "r"(sf) : "memory");
                }
                umma_commit(empty_bar(stage));
                if (++stage == SM_STAGES) { stage = 0; phase ^= 1u; }
            }
            if (ok) umma_commit(tfull_bar);
        }
    } else if (warp < 6) {
        // ---- epilogue: this warp's 32 rows x 32 columns ----
        const int q = warp & 3;
        const int64_t m = (int64_t)m0 + q * 32 + lane;
        // thresholds of this CTA's 32 columns: lane l holds column n0 + l's
        int32_t my_thr = 0; uint32_t my_flip = 0;
        if (p.out_bits != nullptr && n0 + lane < p.N) {
            my_thr = __ldg(p.thr + n0 + lane);
            my_flip = p.flip ? (uint32_t)(__ldg(p.flip + n0 + lane) != 0) : 0u;
        }
        const bool landed = __all_sync(0xffffffffu, mbar_wait(tfull_bar, 0, abort_flag, 23)) != 0;
        if (landed) {
            tc_fence_after();
            int32_t iv[32];
            {
                // the four partial sums are exact integers in fp32, and so is their sum (below 2^24 by the caller's check)
                uint32_t v[32], u[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16), v);
#pragma unroll 1
                for (int a = 1; a < NACC; ++a) {
                    tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * SM_BN), u);
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(u[j]));
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) iv[j] = __float2int_rn(__uint_as_float(v[j]));
            }
            if (p.out != nullptr && m < p.M) {
                int32_t *dst = p.out + m * p.ldo + n0;
                if (n0 + SM_BN <= p.N && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) *reinterpret_cast<int4 *>(dst + j) = make_int4(iv[j], iv[j + 1], iv[j + 2], iv[j + 3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (n0 + j < p.N) dst[j] = iv[j];
                }
            }
            if (p.out_bits != nullptr) {
                // bit j = (sum_j >= thr_j) xor flip_j: column j's threshold comes from lane j
                uint32_t w = 0;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int32_t tj = __shfl_sync(0xffffffffu, my_thr, j);
                    w |= (uint32_t)(iv[j] >= tj) << j;
                }
                const uint32_t fw = __ballot_sync(0xffffffffu, my_flip != 0);
                const int64_t left = p.N - n0;
                const uint32_t nmask = left >= 32 ? 0xffffffffu : ((1u << (int)left) - 1u);
                w = (w ^ fw) & nmask;
                if (m < p.M) p.out_bits[m * p.ld_bits + (n0 >> 5)] = w;
            }
        }
    } else {
        // ---- converters: per operand stage (256 k) the A tile is 128 rows x 8 packed words, the B tile 32 rows x 8 words;
        // item i of a tile is (row i / 8, word i % 8): thread t expands A items t, t + 512 and, if t < 256, B item t.
        // Where an item sits never changes, so its offsets are worked out once; a block that lies wholly inside K and
        // rows inside the matrix take the mask-free path.
        const int t = threadIdx.x - 6 * 32;
        const int word = t & 7;
        int a_src[SM_A_ITEMS], a_dst[SM_A_ITEMS]; bool a_row_ok[SM_A_ITEMS];
#pragma unroll
        for (int i = 0; i < SM_A_ITEMS; ++i) {
            const int row = (t + SM_CONV_THREADS * i) >> 3;
            a_src[i] = row * p.sbw + word;
            a_dst[i] = row * 128 + ((word ^ (row & 7)) << 4);
            a_row_ok[i] = m0 + row < p.M;
        }
        const bool has_b = t < SM_BN * 8;                         // the B tile has 256 words per stage
        const int b_row = (t >> 3) & (SM_BN - 1);
        const int b_src = b_row * p.sbw + word;
        const int sb_blocks = p.sbw * 32 / SM_KB;                // operand stages per packed tile
        const int b_dst = SM_A_BYTES + b_row * 128 + ((word ^ (b_row & 7)) << 4);
        const bool b_row_ok = n0 + b_row < p.N;
        const bool a_signs = p.ka == 1 && p.a_pm1, b_signs = p.kb == 1 && p.b_pm1;      // the common case: one plane of +-1
        int stage = 0; uint32_t phase = 0;
        int buf = 0; uint32_t pphase = 0;
        bool ok = true;
        for (int32_t sb = 0; sb < p.num_sb && ok; ++sb) {
            int landed = 1;
            if (lane == 0) landed = mbar_wait(pfull_bar(buf), pphase, abort_flag, 24) ? 1 : 0;
            landed = __shfl_sync(0xffffffffu, landed, 0);
            if (!landed) { ok = false; break; }
            const uint32_t *pa = reinterpret_cast<const uint32_t *>(gen + packed_off + buf * packed_bytes);
            const uint32_t *pb = reinterpret_cast<const uint32_t *>(gen + packed_off + buf * packed_bytes + p.pa_bytes);
            for (int kbi = 0; kbi < sb_blocks && ok; ++kbi) {
                const int64_t kblock = (int64_t)sb * sb_blocks + kbi;
                if (kblock >= num_kb) break;
                // valid elements of this thread's word (all 32 except in the last words of K)
                const int64_t left = p.K - (kblock * SM_KB + word * 32);
                const uint32_t kvalid = left >= 32 ? 0xffffffffu : (left > 0 ? ((1u << (int)left) - 1u) : 0u);
                // expand first (registers), then wait for the operand stage
                uint4 ea[SM_A_ITEMS], eb = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int i = 0; i < SM_A_ITEMS; ++i) {
                    const uint32_t w0 = pa[a_src[i] + kbi * 8];
                    if (!a_row_ok[i]) ea[i] = make_uint4(0u, 0u, 0u, 0u);
                    else if (a_signs && kvalid == 0xffffffffu) ea[i] = signs_to_fp4_full(w0);
                    else ea[i] = planes_to_fp4(w0, p.ka > 1 ? pa[BM * p.sbw + a_src[i] + kbi * 8] : 0u, p.ka, p.a_pm1, kvalid);
                }
                if (has_b) {
                    const uint32_t w0 = pb[b_src + kbi * 8];
                    if (!b_row_ok) eb = make_uint4(0u, 0u, 0u, 0u);
                    else if (b_signs && kvalid == 0xffffffffu) eb = signs_to_fp4_full(w0);
                    else eb = planes_to_fp4(w0, p.kb > 1 ? pb[SM_BN * p.sbw + b_src + kbi * 8] : 0u, p.kb, p.b_pm1, kvalid);
                }
                // (every lane polls: measured faster than one lane polling and a shuffle)
                if (!__all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 25))) { ok = false; break; }
                uint8_t *at = gen + stage * SM_STAGE_BYTES;
#pragma unroll
                for (int i = 0; i < SM_A_ITEMS; ++i) *reinterpret_cast<uint4 *>(at + a_dst[i]) = ea[i];       // (128-byte swizzle in a_dst)
                if (has_b) *reinterpret_cast<uint4 *>(at + b_dst) = eb;
                fence_async_shared();
                __syncwarp();
                if (lane == 0) mbar_arrive(full_bar(stage));
                if (++stage == SM_STAGES) { stage = 0; phase ^= 1u; }
            }
            __syncwarp();                                        // every lane is done reading this packed tile
            if (lane == 0) mbar_arrive(pempty_bar(buf));
            if (++buf == SM_PACKED_BUFS) { buf = 0; pphase ^= 1u; }
        }
    }

    // ---- teardown ----
    __syncwarp();
    if (*abort_flag) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) tmem_dealloc<1>(tmem_base, TMEM_COLS);
}

// packed planes [planes][rows, ld words] as a 3-D tensor of 32-bit words; box = 64 words x box_rows x 1 plane
int make_packed_map(CUtensorMap *map, const uint32_t *base, int64_t rows, int64_t kwords, int64_t ld, int planes, int64_t plane_stride,
                    int box_rows, int sbw)
{
    EncodeTiledFn fn = encode_fn();
    QNN_REQUIRE(fn != nullptr, QNN_ERR_CUDA, "small-batch gemm: cuTensorMapEncodeTiled is not available from this driver");
    cuuint64_t dims[3] = {(cuuint64_t)kwords, (cuuint64_t)rows, (cuuint64_t)planes};
    cuuint64_t strides[2] = {(cuuint64_t)ld * 4, (cuuint64_t)(planes > 1 ? plane_stride : rows * ld) * 4};
    cuuint32_t box[3] = {(cuuint32_t)sbw, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<uint32_t *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    QNN_REQUIRE(r == CUDA_SUCCESS, QNN_ERR_CUDA, "small-batch gemm: cuTensorMapEncodeTiled failed with code %d", (int)r);
    return QNN_OK;
}

}  // namespace

int smallm_status(int *code)
{
    QNN_CUDA(status_read_clear(code));
    return QNN_OK;
}

// Whether the product can run on the small-batch kernel: packed operands of at most two planes whose sums stay exact in
// fp32, int32 rows and / or thresholded bits as outputs, and rows that TMA can address (16-byte aligned, 16-byte pitch).
// packed words of K per row in one packed tile: 64, or 32 when two tiles of every plane would not fit next to the stages
static int smallm_tile_words(int ka, int kb)
{
    const int packed = (ka * BM + kb * SM_BN) * SM_SB_WORDS * 4;
    return SM_STAGES * SM_STAGE_BYTES + SM_PACKED_BUFS * packed + 256 + 1024 <= SMEM_LIMIT ? SM_SB_WORDS : SM_SB_WORDS / 2;
}

bool gemm_smallm_supported(const GemmArgs &g)
{
    if (g.a_tc || g.b_tc || g.out_form || g.conv || !g.a || !g.b) return false;
    if (g.epilogue != EPI_ROWMAJOR && g.epilogue != EPI_BITS) return false;
    if (g.kwords > 0 && g.kwords != ceil_div(g.K, 32)) return false;
    if (g.K < 1 || tc_pick_form(g.ka, g.a_mode, g.kb, g.b_mode, g.K) != QNN_FORM_FP4) return false;
    if (!aligned(g.a, 16) || !aligned(g.b, 16) || g.lda % 4 != 0 || g.ldb % 4 != 0) return false;
    if (g.ka > 1 && g.a_plane_stride % 4 != 0) return false;
    if (g.kb > 1 && g.b_plane_stride % 4 != 0) return false;
    if (ceil_div(g.N, SM_BN) > 0x7fffffff || ceil_div(g.M, BM) > 65535) return false;
    return true;
}

int launch_gemm_smallm(const GemmArgs &g, cudaStream_t st)
{
    QNN_REQUIRE(gemm_smallm_supported(g), QNN_ERR_UNSUPPORTED, "small-batch gemm: operands or outputs not supported by this kernel");
    const int64_t kwords = ceil_div(g.K, 32);
    SmParams p{};
    p.M = g.M; p.N = g.N; p.K = g.K;
    p.sbw = smallm_tile_words(g.ka, g.kb);
    p.num_sb = (int32_t)ceil_div(kwords, p.sbw);
    p.ka = g.ka; p.kb = g.kb; p.a_pm1 = g.a_mode == QNN_MODE_PM1; p.b_pm1 = g.b_mode == QNN_MODE_PM1;
    p.pa_bytes = g.ka * BM * p.sbw * 4;
    p.pb_bytes = g.kb * SM_BN * p.sbw * 4;
    p.out = g.out; p.ldo = g.ldo; p.thr = g.thr; p.flip = g.flip; p.out_bits = g.out_bits; p.ld_bits = g.ld_bits;
    p.idesc = (1u << 7) | (1u << 10) | (1u << 23) | ((uint32_t)(BM >> 4) << 24) | ((uint32_t)(SM_BN >> 3) << 17);
    CUtensorMap ma, mb;
    if (int rc = make_packed_map(&ma, g.a, g.M, kwords, g.lda, g.ka, g.a_plane_stride, BM, p.sbw)) return rc;
    if (int rc = make_packed_map(&mb, g.b, g.N, kwords, g.ldb, g.kb, g.b_plane_stride, SM_BN, p.sbw)) return rc;
    const int smem = SM_STAGES * SM_STAGE_BYTES + SM_PACKED_BUFS * (p.pa_bytes + p.pb_bytes) + 256 + 1024;
    QNN_REQUIRE(smem <= SMEM_LIMIT, QNN_ERR_UNSUPPORTED, "small-batch gemm: packed tiles do not fit shared memory");
    static std::atomic<int> opted_in[64];                 // largest shared-memory size asked for so far, per device
    int dev = 0;
    QNN_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || opted_in[dev].load(std::memory_order_acquire) < smem) {
        QNN_CUDA(cudaFuncSetAttribute(gemm_smallm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT));
        if (dev >= 0 && dev < 64) opted_in[dev].store(SMEM_LIMIT, std::memory_order_release);
    }
    profile_before(st);
    QNN_CUDA(launch_pdl(gemm_smallm_kernel, dim3((unsigned)ceil_div(g.N, SM_BN), (unsigned)ceil_div(g.M, BM)), dim3(SM_THREADS), (size_t)smem, st,
                        ma, mb, p));
    profile_after(st);
    return check_launch("small-batch gemm");
}

}  // namespace qnn
