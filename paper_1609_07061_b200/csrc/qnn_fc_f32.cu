// A binary fully-connected layer whose weights are still real-valued, in ONE pass over them:
//     out[m, n] = sum_k sign(x[m, k]) * sign(w[k, n])          (Eq. 1 on both operands, Algorithm 4's hidden-layer product)
// For a small batch every weight is used by a single 128-row tile, so nothing is gained by first writing packed
// weights and reading them back: the 4 bytes per weight that have to come from HBM anyway are all the traffic
// there is.  Converter warps read w[K, N] (coalesced along n), apply Eq. 1 and write the +-1 values as e2m1 nibbles
// straight into the 128-byte-swizzled shared-memory tile that tcgen05.mma reads as its B operand; the activations
// (already in e2m1 form, a few hundred KB) arrive through TMA; one thread issues the block-scaled e2m1 products with
// unit scales, fp32 accumulation in tensor memory (exact integers below 2^24); four warps write the int32 result.
//
//   warp 0        TMA: A tiles (128 rows x 128 bytes of K per stage)
//   warp 1        tcgen05.mma issue, tensor-memory owner
//   warps 2..5    epilogue: tcgen05.ld -> int32 rows
//   warps 6..     converters (16 warps; 8 on the register path): fp32 weights -> e2m1 B tile (32 output units x 256 k per stage)
//
// Every device-side wait is bounded (status word, clean exit), as in the product kernel.
#include <atomic>
#include "qnn_internal.cuh"
#include "qnn_tc_ptx.cuh"

namespace qnn {
namespace {

constexpr int FC_BN = 32;                      // output units per CTA
constexpr int FC_KB = 256;                     // k per pipeline stage (128 bytes of e2m1)
// converter warps: 16 when the weights arrive as TMA tiles (four k per thread; the kernel is bound by the converters'
// instruction stream, and twice the warps hide twice the latency), 8 on the register path (eight k per thread)
constexpr int fc_threads(int cw) { return 32 * (6 + cw); }
constexpr int FC_A_BYTES = BM * BKB;           // 16 KB
constexpr int FC_B_BYTES = FC_BN * BKB;        // 4 KB
constexpr int FC_STAGE_BYTES = FC_A_BYTES + FC_B_BYTES;
constexpr int FC_STAGES = 3;                   // operand stages (e2m1 A tile + converted B tile)
constexpr int FC_W_BYTES = FC_KB * FC_BN * 4;  // 32 KB: one K block of this CTA's fp32 weight columns
constexpr int FC_W_STAGES = 5;                 // fp32 weight tiles in flight (TMA): 160 KB per SM -- the kernel lives on these
constexpr int FC_W_OFFSET = FC_STAGES * FC_STAGE_BYTES;
constexpr int FC_BAR_OFFSET = FC_W_OFFSET + FC_W_STAGES * FC_W_BYTES;
constexpr int FC_SMEM = FC_BAR_OFFSET + 256 + 1024;

struct FcParams {
    const float *w; int64_t ldw;
    int64_t M, N, K;
    int32_t num_kb;
    int32_t *out; int64_t ldo;
    uint32_t idesc;
    int vec;                                   // weights allow 16-byte loads
    int w_tma;                                 // weights arrive as TMA boxes in shared memory (else: loads into registers)
};

__device__ __forceinline__ uint32_t sign_nibble(float v) { return v >= 0.0f ? 0x2u : 0xAu; }   // +1 / -1 as e2m1

template <int CW, bool WTMA>
__global__ void __launch_bounds__(fc_threads(CW), 1)
fc_sign_f32_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w, const FcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - raw);
    const uint32_t bar0 = base + FC_BAR_OFFSET;
    uint64_t *bars = reinterpret_cast<uint64_t *>(gen + FC_BAR_OFFSET);
    auto full_bar = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (uint32_t)(FC_STAGES + s); };
    const uint32_t tfull_bar = bar0 + 8u * (uint32_t)(2 * FC_STAGES);
    auto wfull_bar = [&](int s) { return bar0 + 8u * (uint32_t)(2 * FC_STAGES + 1 + s); };
    auto wempty_bar = [&](int s) { return bar0 + 8u * (uint32_t)(2 * FC_STAGES + 1 + FC_W_STAGES + s); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * FC_STAGES + 1 + 2 * FC_W_STAGES);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int64_t n0 = (int64_t)blockIdx.x * FC_BN;
    const int32_t m0 = (int32_t)blockIdx.y * BM;
    griddep_launch_dependents();

    if (threadIdx.x == 0) {
        // a stage is full when the TMA bytes have landed AND every converter warp has written its part
        for (int s = 0; s < FC_STAGES; ++s) { mbar_init(full_bar(s), 1 + CW); mbar_init(empty_bar(s), 1); }
        mbar_init(tfull_bar, 1);
        for (int s = 0; s < FC_W_STAGES; ++s) { mbar_init(wfull_bar(s), 1); mbar_init(wempty_bar(s), CW); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // The four K steps of a stage go to FOUR accumulators, added in the epilogue: at 32 columns a product is far shorter
    // than the pipe's latency, and a single accumulator would make every product wait for the one before it.
    constexpr int NACC = 4;
    constexpr uint32_t SCALE_COL = NACC * FC_BN;
    constexpr uint32_t TMEM_COLS = 256;
    if (warp == 1) tmem_alloc<1>(smem_u32(tmem_slot), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (warp >= 2 && warp < 6) {
        // unit scale factors (ue8m0 exponent 127) in every lane of the scale columns
        const int q = warp & 3;
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_st8(tmem_base + ((uint32_t)(q * 32) << 16) + SCALE_COL + (uint32_t)(8 * c), 0x7f7f7f7fu);
        tmem_st_wait();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    // the activations were written by the kernel before this one; the weights were not
    if (warp == 0) {
        if (lane == 0) {
            // Two rings: fp32 weight tiles (32 columns x 256 k, 32 KB each, as many in flight as fit) and the A tiles of the
            // operand stages.  The weights do not depend on the kernel before this one, the activations do: the first
            // weight tiles are on their way before the dependency wait.
            int ws = 0; uint32_t wphase = 0; int32_t wkb = 0;
            auto issue_w = [&]() -> bool {
                if (!mbar_wait(wempty_bar(ws), wphase ^ 1u, abort_flag, 15)) return false;
                asm volatile(
                    "mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n"
                    "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%2], [%3, {%4, %5}], [%0];\n"
                    ::"r"(wfull_bar(ws)), "r"((uint32_t)FC_W_BYTES), "r"(base + (uint32_t)(FC_W_OFFSET + ws * FC_W_BYTES)), "l"(&tmap_w),
                      "r"((int32_t)n0), "r"(wkb * FC_KB) : "memory");
                ++wkb;
                if (++ws == FC_W_STAGES) { ws = 0; wphase ^= 1u; }
                return true;
            };
            bool ok = true;
            if (WTMA)
                while (ok && wkb < p.num_kb && wkb < FC_W_STAGES) ok = issue_w();
            griddep_wait();
            int stage = 0; uint32_t phase = 0;
            for (int32_t kb = 0; kb < p.num_kb && ok; ++kb) {
                if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 11)) break;
                asm volatile(
                    "mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n"
                    "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%2], [%3, {%4, %5}], [%0];\n"
                    ::"r"(full_bar(stage)), "r"((uint32_t)FC_A_BYTES), "r"(base + (uint32_t)(stage * FC_STAGE_BYTES)), "l"(&tmap_a),
                      "r"(kb * BKB), "r"(m0) : "memory");
                if (++stage == FC_STAGES) { stage = 0; phase ^= 1u; }
                if (WTMA && wkb < p.num_kb) ok = issue_w();
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            const uint32_t sf = tmem_base + SCALE_COL;
            for (int32_t kb = 0; kb < p.num_kb && ok; ++kb) {
                if (!mbar_wait(full_bar(stage), phase, abort_flag, 12)) { ok = false; break; }
                tc_fence_after();
                const uint32_t sa = base + (uint32_t)(stage * FC_STAGE_BYTES);
                const uint64_t da = make_kmajor_desc<BKB>(sa), db = make_kmajor_desc<BKB>(sa + FC_A_BYTES);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint64_t a = da + (uint64_t)(2 * ks), b = db + (uint64_t)(2 * ks);
                    const uint32_t acc = kb != 0;
                    asm volatile("{\n.reg .pred P;\nsetp.ne.b32 P, %4, 0;\n"
                                 "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%5], P;\n}\n"
                                 ::"r"(tmem_base + (uint32_t)(ks * FC_BN)), "l"(a), "l"(b), "r"(p.idesc), "r"(acc), "r"(sf) : "memory");
                }
                umma_commit(empty_bar(stage));                 // the stage is free again once these products have run
                if (++stage == FC_STAGES) { stage = 0; phase ^= 1u; }
            }
            if (ok) umma_commit(tfull_bar);
        }
    } else if (warp < 6) {
        // ---- epilogue: this warp's 32 rows of the accumulator -> int32 ----
        const int q = warp & 3;
        const bool landed = __all_sync(0xffffffffu, mbar_wait(tfull_bar, 0, abort_flag, 13)) != 0;
        if (landed) {
            tc_fence_after();
            griddep_wait();                              // (returns at once here: the activations' producer has long finished)
            uint32_t v[32];
            {
                uint32_t u[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16), v);
#pragma unroll 1
                for (int a = 1; a < NACC; ++a) {
                    tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * FC_BN), u);
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) + __uint_as_float(u[j]));
                }
            }
            const int64_t m = (int64_t)m0 + q * 32 + lane;
            if (m < p.M) {
                int32_t *dst = p.out + m * p.ldo + n0;
                if (n0 + FC_BN <= p.N && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<int4 *>(dst + j) = make_int4(__float2int_rn(__uint_as_float(v[j])), __float2int_rn(__uint_as_float(v[j + 1])),
                                                                       __float2int_rn(__uint_as_float(v[j + 2])), __float2int_rn(__uint_as_float(v[j + 3])));
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (n0 + j < p.N) dst[j] = __float2int_rn(__uint_as_float(v[j]));
                }
            }
        }
    } else {
        // ---- converters: thread (cw, lane) owns columns n0 + 4*(lane & 7) .. +3 and the KPT consecutive k of group
        // kq = cw*4 + (lane >> 3) in every K block; a warp's load of one k row set is 4 rows x 128 contiguous bytes.
        constexpr int KPT = FC_KB / (4 * CW);                    // k per thread and block: 8 or 4
        const int cw = warp - 6;
        const int n4 = lane & 7;
        const int kq = cw * 4 + (lane >> 3);
        const int64_t ncol = n0 + 4 * n4;
        const bool cols_ok = ncol + 4 <= p.N;
        int stage = 0; uint32_t phase = 0;
        const bool ragged_cols = n0 + FC_BN > p.N;
        // KPT k x four columns of fp32 weights -> four words of KPT e2m1 nibbles; what lies outside the matrix -> 0
        auto convert = [&](const float4 (&t)[KPT], int32_t kb, uint32_t (&wv)[4]) {
            const bool ragged = ragged_cols || ((int64_t)(kb + 1) * FC_KB > p.K);       // (uniform over the CTA)
            if (!ragged) {
                // the common case, kept free of any index test: a compare, a select and a shifted OR per element
                // (0xA = -1, flipped to 0x2 = +1 where x >= 0)
#pragma unroll
                for (int c = 0; c < 4; ++c) wv[c] = KPT == 8 ? 0xAAAAAAAAu : 0xAAAAu;
#pragma unroll
                for (int j = 0; j < KPT; ++j) {
                    wv[0] ^= (t[j].x >= 0.0f ? 8u : 0u) << (4 * j);
                    wv[1] ^= (t[j].y >= 0.0f ? 8u : 0u) << (4 * j);
                    wv[2] ^= (t[j].z >= 0.0f ? 8u : 0u) << (4 * j);
                    wv[3] ^= (t[j].w >= 0.0f ? 8u : 0u) << (4 * j);
                }
                return;
            }
            wv[0] = wv[1] = wv[2] = wv[3] = 0u;
#pragma unroll
            for (int j = 0; j < KPT; ++j) {
                const float e[4] = {t[j].x, t[j].y, t[j].z, t[j].w};
                const bool k_in = (int64_t)kb * FC_KB + kq * KPT + j < p.K;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t nib = sign_nibble(e[c]);
                    if (!(k_in && ncol + c < p.N)) nib = 0u;
                    wv[c] |= nib << (4 * j);
                }
            }
        };
        // writes this thread's words of the B tile of `stage` once the slot is free, then reports the warp's part done
        auto deliver = [&](const uint32_t (&wv)[4]) -> bool {
            // (every lane polls: measured faster than one lane polling and a shuffle)
            if (!__all_sync(0xffffffffu, mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, 14))) return false;
            uint8_t *bt = gen + stage * FC_STAGE_BYTES + FC_A_BYTES;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int row = 4 * n4 + c;
                // 128-byte swizzle: 16-byte chunk index XOR (row mod 8); this thread's KPT/2 bytes sit at byte kq*KPT/2 of the row
                const int off = kq * (KPT / 2);
                uint8_t *dstp = bt + row * 128 + (((off >> 4) ^ (row & 7)) << 4) + (off & 15);
                if (KPT == 8) *reinterpret_cast<uint32_t *>(dstp) = wv[c];
                else *reinterpret_cast<uint16_t *>(dstp) = (uint16_t)wv[c];
            }
            fence_async_shared();                                  // generic-proxy writes -> visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(full_bar(stage));
            if (++stage == FC_STAGES) { stage = 0; phase ^= 1u; }
            return true;
        };
        if (WTMA) {
            // weights arrive as [256 k][32 columns] fp32 tiles in shared memory
            int ws = 0; uint32_t wphase = 0;
            bool ok = true;
            for (int32_t kb = 0; kb < p.num_kb && ok; ++kb) {
                int landed = 1;
                if (lane == 0) landed = mbar_wait(wfull_bar(ws), wphase, abort_flag, 16) ? 1 : 0;
                landed = __shfl_sync(0xffffffffu, landed, 0);
                if (!landed) { ok = false; break; }
                const float *wt = reinterpret_cast<const float *>(gen + FC_W_OFFSET + ws * FC_W_BYTES);
                float4 t[KPT];
#pragma unroll
                for (int j = 0; j < KPT; ++j) t[j] = *reinterpret_cast<const float4 *>(wt + (kq * KPT + j) * FC_BN + 4 * n4);
                uint32_t wv[4];
                convert(t, kb, wv);
                __syncwarp();                                        // every lane holds its values in registers: the tile may be refilled
                if (lane == 0) mbar_arrive(wempty_bar(ws));
                if (++ws == FC_W_STAGES) { ws = 0; wphase ^= 1u; }
                ok = deliver(wv);
            }
        } else {
        // (weights that allow no bulk copies: loads into registers)
        // Three K blocks of this thread's weights are in flight at any time (24 x 16 bytes per thread, 96 KB per SM):
        // the kernel lives on the bytes it keeps in flight, a block's registers are refilled as soon as they are consumed.
        constexpr int DEPTH = 3;
        float4 buf[DEPTH][KPT];
        auto load_block = [&](int32_t kb, float4 (&t)[KPT]) {
            const int64_t k0 = (int64_t)kb * FC_KB + kq * KPT;
#pragma unroll
            for (int j = 0; j < KPT; ++j) {
                const int64_t k = k0 + j;
                if (p.vec && cols_ok && k < p.K) {
                    t[j] = __ldcs(reinterpret_cast<const float4 *>(p.w + k * p.ldw + ncol));
                } else {
                    // ragged edges or unaligned weights: element by element (what lies outside the matrix is masked below)
                    float e[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) e[c] = (k < p.K && ncol + c < p.N) ? p.w[k * p.ldw + ncol + c] : 0.0f;
                    t[j] = make_float4(e[0], e[1], e[2], e[3]);
                }
            }
        };
#pragma unroll
        for (int i = 0; i < DEPTH; ++i)
            if (i < p.num_kb) load_block(i, buf[i]);
        bool ok = true;
        for (int32_t kb0 = 0; kb0 < p.num_kb && ok; kb0 += DEPTH) {
#pragma unroll
            for (int i = 0; i < DEPTH; ++i) {
                const int32_t kb = kb0 + i;
                if (kb >= p.num_kb || !ok) break;
                uint32_t wv[4];
                convert(buf[i], kb, wv);
                if (kb + DEPTH < p.num_kb) load_block(kb + DEPTH, buf[i]);
                ok = deliver(wv);
            }
        }
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

}  // namespace

int fc_f32_status(int *code)
{
    QNN_CUDA(status_read_clear(code));
    return QNN_OK;
}

}  // namespace qnn

using namespace qnn;

extern "C" {

size_t qnn_fc_sign_f32_workspace_bytes(int64_t M, int64_t K)
{
    if (M <= 0 || K <= 0) return 0;
    return round_up((size_t)M * (size_t)tc_row_pitch(ceil_div(K, 32), QNN_FORM_FP4), 256);
}

int qnn_fc_sign_f32(const float *x, int64_t M, int64_t K, int64_t ldx, const float *w, int64_t N, int64_t ldw, int32_t *out,
                    int64_t ldo, void *ws, size_t ws_bytes, void *stream)
{
    const char *what = "qnn_fc_sign_f32";
    QNN_REQUIRE(M >= 0 && N >= 0 && K >= 0, QNN_ERR_INVALID_ARG, "%s: negative size", what);
    if (M == 0 || N == 0) return QNN_OK;
    QNN_REQUIRE(K >= 1, QNN_ERR_UNSUPPORTED, "%s: K must be at least 1", what);
    QNN_REQUIRE(K < ((int64_t)1 << 24), QNN_ERR_UNSUPPORTED, "%s: K must be below 2^24 (fp32 accumulation of +-1 products stays exact)", what);
    QNN_REQUIRE(x && w && out, QNN_ERR_INVALID_ARG, "%s: NULL pointer", what);
    QNN_REQUIRE(ldx >= K && ldw >= N && ldo >= N, QNN_ERR_INVALID_ARG, "%s: leading dimension too small", what);
    QNN_REQUIRE(aligned(x, 4) && aligned(w, 4) && aligned(out, 4), QNN_ERR_ALIGNMENT, "%s: pointers must be 4-byte aligned", what);
    QNN_REQUIRE(ceil_div(N, FC_BN) <= 0x7fffffff && ceil_div(M, BM) <= 65535, QNN_ERR_UNSUPPORTED, "%s: shape too large for the launch grid", what);
    const size_t need = qnn_fc_sign_f32_workspace_bytes(M, K);
    QNN_REQUIRE(ws != nullptr && aligned(ws, 256) && ws_bytes >= need, QNN_ERR_WORKSPACE,
                "%s: workspace of at least %zu bytes (256-byte aligned) required", what, need);
    cudaStream_t st = as_stream(stream);
    const int64_t kwords = ceil_div(K, 32);
    const int64_t pitch = tc_row_pitch(kwords, QNN_FORM_FP4);
    CUtensorMap ma;
    {
        EncodeTiledFn fn = encode_fn();
        QNN_REQUIRE(fn != nullptr, QNN_ERR_CUDA, "%s: cuTensorMapEncodeTiled is not available from this driver", what);
        cuuint64_t dims[2] = {(cuuint64_t)tc_row_bytes(kwords, QNN_FORM_FP4), (cuuint64_t)M};
        cuuint64_t strides[1] = {(cuuint64_t)pitch};
        cuuint32_t box[2] = {(cuuint32_t)BKB, (cuuint32_t)BM};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = fn(&ma, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, ws, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        QNN_REQUIRE(r == CUDA_SUCCESS, QNN_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed with code %d", what, (int)r);
    }
    // activations: Eq. 1 straight into e2m1 form (a small kernel; the product kernel's prologue overlaps its tail)
    if (int rc = qnn_quantize_form_sign(x, M, K, ldx, QNN_FORM_FP4, ws, pitch, stream)) return rc;

    FcParams p{};
    p.w = w; p.ldw = ldw; p.M = M; p.N = N; p.K = K;
    CUtensorMap mw = ma;
    p.w_tma = ((ldw % 4 == 0) && aligned(w, 16)) ? 1 : 0;
    if (p.w_tma) {
        // fp32 weights [K, N]: boxes of 32 columns x 256 k, dense in shared memory; reads past either extent give 0
        EncodeTiledFn fn = encode_fn();
        cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)K};
        cuuint64_t strides[1] = {(cuuint64_t)ldw * 4};
        cuuint32_t box[2] = {(cuuint32_t)FC_BN, (cuuint32_t)FC_KB};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = fn(&mw, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(w), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        QNN_REQUIRE(r == CUDA_SUCCESS, QNN_ERR_CUDA, "%s: cuTensorMapEncodeTiled (weights) failed with code %d", what, (int)r);
    }
    p.num_kb = (int32_t)ceil_div(K, FC_KB);
    p.out = out; p.ldo = ldo;
    p.idesc = (1u << 7) | (1u << 10) | (1u << 23) | ((uint32_t)(BM >> 4) << 24) | ((uint32_t)(FC_BN >> 3) << 17);
    p.vec = (ldw % 4 == 0) && aligned(w, 16);
    static std::atomic<bool> opted_in[64];
    int dev = 0;
    QNN_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !opted_in[dev].load(std::memory_order_acquire)) {
        QNN_CUDA(cudaFuncSetAttribute(fc_sign_f32_kernel<16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FC_SMEM));
        QNN_CUDA(cudaFuncSetAttribute(fc_sign_f32_kernel<8, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FC_SMEM));
        if (dev >= 0 && dev < 64) opted_in[dev].store(true, std::memory_order_release);
    }
    const dim3 grid((unsigned)ceil_div(N, FC_BN), (unsigned)ceil_div(M, BM));
    if (p.w_tma)
        QNN_CUDA(launch_pdl(fc_sign_f32_kernel<16, true>, grid, dim3(fc_threads(16)), (size_t)FC_SMEM, st, ma, mw, p));
    else
        QNN_CUDA(launch_pdl(fc_sign_f32_kernel<8, false>, grid, dim3(fc_threads(8)), (size_t)FC_SMEM, st, ma, mw, p));
    return check_launch(what);
}

}  // extern "C"
