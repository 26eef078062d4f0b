// Tensor-core matrix product on the 5th-generation tensor cores (tcgen05).
//
// The packed bit-planes are first rewritten in a "tensor-core form", one VALUE
// per element (+-1, unsigned codes or signed-symmetric codes; pad positions 0):
//   QNN_FORM_FP4  4-bit e2m1 floats, two per byte -- holds {0, +-1, +-2, +-3};
//                 multiplied by tcgen05.mma kind::mxf4 with all block scales 1.0
//                 and accumulated in fp32, which is exact for these integers
//                 while |sum| < 2^24;
//   QNN_FORM_I8   int8 / uint8 -- any code that fits a byte; kind::i8, int32
//                 accumulation.
// One multiply-accumulate of the tensor core carries one product of the
// paper's sum, so a k-bit x k-bit product costs ONE pass here instead of ka*kb
// plane passes.  A persistent, warp-specialised kernel does the product:
//   warp 0: TMA (128-byte swizzle) -> shared-memory ring
//   warp 1: tcgen05.mma, accumulator in tensor memory (two accumulator stages)
//   warps 2..5: tcgen05.ld epilogue -> int32 rows, NCHW scatter, threshold ->
//               packed bits and / or the next layer's operand in tensor-core form
// A convolution can be run as an implicit GEMM: the A tile of one filter tap is
// a 4-D TMA box of the NHWC tensor, out-of-image reads give zero, and the
// contribution of the padding value is added back per border class.
//
// Every device-side wait is bounded: when a wait runs out the kernel records a
// code in a device status word, raises a block-wide abort flag, lets copies in
// flight land, frees its tensor memory and returns.
#include <cuda.h>
#include <atomic>
#include <cstdlib>
#include "qnn_internal.cuh"
#include "qnn_tc_ptx.cuh"

namespace qnn {
namespace {

constexpr int EPI_GROUPS = 2;        // epilogue warps per quarter of the accumulator's lanes
constexpr int tc_threads(int groups) { return 64 + 128 * groups; }   // warp 0: TMA, warp 1: MMA + TMEM owner, the rest: epilogue
constexpr int TC_THREADS = tc_threads(EPI_GROUPS);

struct TcParams {
    int64_t M, N;
    int32_t num_kb;                  // K blocks of BKB bytes
    int32_t tiles_m, tiles_n;
    int32_t a_tx_bytes;              // bytes one A box delivers
    int epilogue;
    int32_t *out; int64_t ldo; int64_t hw;
    const int32_t *thr; const uint8_t *flip; uint32_t *out_bits; int64_t ld_bits;
    uint8_t *out_form; int64_t ld_form; int out_form_kind;
    uint32_t idesc;
    // The last column block may be narrower than the tile: its instructions then multiply only n_last columns
    // (a multiple of 16), described by idesc_last, and a pair's second CTA loads its B rows n_last / 2 further on.
    uint32_t idesc_last; int32_t n_last;
    int32_t thr_clamp;               // int8 form: max |sum| + 1 when that is below 2^30 (else 0: plain compares)
    // asynchronous (TMA) stores through the per-warp staging buffers: 0 = plain stores from registers
    int tma_out;                     // 1: int32 row-major [M, N]; 2: int32 NCHW [img, n, pix]
    // implicit convolution (conv != 0)
    int conv;
    int32_t cH, cW, cR, tiles_per_img, cKW, cpad, cblocks;
    int32_t cG, cB;             // images per tile (> 1 only when a whole image is at most half a tile), images in all
    int32_t pool;               // conv: 2 x 2 max-pooling of the thresholded signs inside the epilogue
    const int32_t *corr;
    int64_t corr_ld;                 // row length of the correction table: N rounded up to 32, pad zero
};

// One pipeline stage of the MMA warp as ONE instruction stream: poll the NEXT stage's full barrier, issue the
// four K steps of this stage (+32 bytes of K = +2 in the descriptors' address field), commit them to this
// stage's empty barrier, and only then read the poll's result -- the poll's latency hides behind the issue.
// Returns non-zero when the next stage has already landed.
template <int FORM>
__device__ __forceinline__ uint32_t umma_stage(uint32_t next_full_bar, uint32_t next_parity, uint32_t d_tmem, uint32_t a_lo,
                                               uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t accumulate_first,
                                               uint32_t sf, uint32_t empty_bar)
{
    uint32_t ready;
    if (FORM == QNN_FORM_FP4) {
        asm volatile(
            "{\n"
            ".reg .pred P, Q, T;\n"
            ".reg .b64 a0, a1, a2, a3, b0, b1, b2, b3;\n"
            ".reg .b32 t1, t2, t3, u1, u2, u3;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 Q, [%1], %2;\n"
            "setp.ne.b32 P, %7, 0;\n"
            "setp.eq.b32 T, 0, 0;\n"
            "add.u32 t1, %4, 2;\n add.u32 t2, %4, 4;\n add.u32 t3, %4, 6;\n"
            "add.u32 u1, %5, 2;\n add.u32 u2, %5, 4;\n add.u32 u3, %5, 6;\n"
            "mov.b64 a0, {%4, %10};\n mov.b64 a1, {t1, %10};\n mov.b64 a2, {t2, %10};\n mov.b64 a3, {t3, %10};\n"
            "mov.b64 b0, {%5, %10};\n mov.b64 b1, {u1, %10};\n mov.b64 b2, {u2, %10};\n mov.b64 b3, {u3, %10};\n"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%3], a0, b0, %6, [%8], [%8], P;\n"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%3], a1, b1, %6, [%8], [%8], T;\n"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%3], a2, b2, %6, [%8], [%8], T;\n"
            "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%3], a3, b3, %6, [%8], [%8], T;\n"
            "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%9];\n"
            "selp.u32 %0, 1, 0, Q;\n"
            "}\n"
            : "=r"(ready)
            : "r"(next_full_bar), "r"(next_parity), "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate_first),
              "r"(sf), "r"(empty_bar), "r"(desc_hi)
            : "memory");
    } else {
        asm volatile(
            "{\n"
            ".reg .pred P, Q, T;\n"
            ".reg .b64 a0, a1, a2, a3, b0, b1, b2, b3;\n"
            ".reg .b32 t1, t2, t3, u1, u2, u3;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 Q, [%1], %2;\n"
            "setp.ne.b32 P, %7, 0;\n"
            "setp.eq.b32 T, 0, 0;\n"
            "add.u32 t1, %4, 2;\n add.u32 t2, %4, 4;\n add.u32 t3, %4, 6;\n"
            "add.u32 u1, %5, 2;\n add.u32 u2, %5, 4;\n add.u32 u3, %5, 6;\n"
            "mov.b64 a0, {%4, %10};\n mov.b64 a1, {t1, %10};\n mov.b64 a2, {t2, %10};\n mov.b64 a3, {t3, %10};\n"
            "mov.b64 b0, {%5, %10};\n mov.b64 b1, {u1, %10};\n mov.b64 b2, {u2, %10};\n mov.b64 b3, {u3, %10};\n"
            "tcgen05.mma.cta_group::1.kind::i8 [%3], a0, b0, %6, P;\n"
            "tcgen05.mma.cta_group::1.kind::i8 [%3], a1, b1, %6, T;\n"
            "tcgen05.mma.cta_group::1.kind::i8 [%3], a2, b2, %6, T;\n"
            "tcgen05.mma.cta_group::1.kind::i8 [%3], a3, b3, %6, T;\n"
            "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%9];\n"
            "selp.u32 %0, 1, 0, Q;\n"
            "}\n"
            : "=r"(ready)
            : "r"(next_full_bar), "r"(next_parity), "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate_first),
              "r"(sf), "r"(empty_bar), "r"(desc_hi)
            : "memory");
    }
    return ready;
}

// The stage of a 64-byte K block (e2m1, single CTA): two K steps.
__device__ __forceinline__ uint32_t umma_stage_half(uint32_t next_full_bar, uint32_t next_parity, uint32_t d_tmem, uint32_t a_lo,
                                                    uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t accumulate_first,
                                                    uint32_t sf, uint32_t empty_bar)
{
    uint32_t ready;
    asm volatile(
        "{\n"
        ".reg .pred P, Q, T;\n"
        ".reg .b64 a0, a1, b0, b1;\n"
        ".reg .b32 t1, u1;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 Q, [%1], %2;\n"
        "setp.ne.b32 P, %7, 0;\n"
        "setp.eq.b32 T, 0, 0;\n"
        "add.u32 t1, %4, 2;\n add.u32 u1, %5, 2;\n"
        "mov.b64 a0, {%4, %10};\n mov.b64 a1, {t1, %10};\n mov.b64 b0, {%5, %10};\n mov.b64 b1, {u1, %10};\n"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%3], a0, b0, %6, [%8], [%8], P;\n"
        "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%3], a1, b1, %6, [%8], [%8], T;\n"
        "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%9];\n"
        "selp.u32 %0, 1, 0, Q;\n"
        "}\n"
        : "=r"(ready)
        : "r"(next_full_bar), "r"(next_parity), "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate_first),
          "r"(sf), "r"(empty_bar), "r"(desc_hi)
        : "memory");
    return ready;
}

// The same stage for a CTA pair (issued by the leader CTA): one instruction multiplies the 256 x BN tile of both
// CTAs; the commit arrives on this stage's empty barrier of BOTH CTAs.
template <int FORM>
__device__ __forceinline__ uint32_t umma_stage_pair(uint32_t next_full_bar, uint32_t next_parity, uint32_t d_tmem, uint32_t a_lo,
                                                    uint32_t b_lo, uint32_t desc_hi, uint32_t idesc, uint32_t accumulate_first,
                                                    uint32_t sf, uint32_t empty_bar)
{
    uint32_t ready;
    if (FORM == QNN_FORM_FP4) {
        asm volatile(
            "{\n"
            ".reg .pred P, Q, T;\n"
            ".reg .b64 a0, a1, a2, a3, b0, b1, b2, b3;\n"
            ".reg .b32 t1, t2, t3, u1, u2, u3;\n"
            ".reg .b16 both;\n"
            "mov.b16 both, 3;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 Q, [%1], %2;\n"
            "setp.ne.b32 P, %7, 0;\n"
            "setp.eq.b32 T, 0, 0;\n"
            "add.u32 t1, %4, 2;\n add.u32 t2, %4, 4;\n add.u32 t3, %4, 6;\n"
            "add.u32 u1, %5, 2;\n add.u32 u2, %5, 4;\n add.u32 u3, %5, 6;\n"
            "mov.b64 a0, {%4, %10};\n mov.b64 a1, {t1, %10};\n mov.b64 a2, {t2, %10};\n mov.b64 a3, {t3, %10};\n"
            "mov.b64 b0, {%5, %10};\n mov.b64 b1, {u1, %10};\n mov.b64 b2, {u2, %10};\n mov.b64 b3, {u3, %10};\n"
            "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%3], a0, b0, %6, [%8], [%8], P;\n"
            "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%3], a1, b1, %6, [%8], [%8], T;\n"
            "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%3], a2, b2, %6, [%8], [%8], T;\n"
            "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%3], a3, b3, %6, [%8], [%8], T;\n"
            "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%9], both;\n"
            "selp.u32 %0, 1, 0, Q;\n"
            "}\n"
            : "=r"(ready)
            : "r"(next_full_bar), "r"(next_parity), "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate_first),
              "r"(sf), "r"(empty_bar), "r"(desc_hi)
            : "memory");
    } else {
        asm volatile(
            "{\n"
            ".reg .pred P, Q, T;\n"
            ".reg .b64 a0, a1, a2, a3, b0, b1, b2, b3;\n"
            ".reg .b32 t1, t2, t3, u1, u2, u3;\n"
            ".reg .b16 both;\n"
            "mov.b16 both, 3;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 Q, [%1], %2;\n"
            "setp.ne.b32 P, %7, 0;\n"
            "setp.eq.b32 T, 0, 0;\n"
            "add.u32 t1, %4, 2;\n add.u32 t2, %4, 4;\n add.u32 t3, %4, 6;\n"
            "add.u32 u1, %5, 2;\n add.u32 u2, %5, 4;\n add.u32 u3, %5, 6;\n"
            "mov.b64 a0, {%4, %10};\n mov.b64 a1, {t1, %10};\n mov.b64 a2, {t2, %10};\n mov.b64 a3, {t3, %10};\n"
            "mov.b64 b0, {%5, %10};\n mov.b64 b1, {u1, %10};\n mov.b64 b2, {u2, %10};\n mov.b64 b3, {u3, %10};\n"
            "tcgen05.mma.cta_group::2.kind::i8 [%3], a0, b0, %6, P;\n"
            "tcgen05.mma.cta_group::2.kind::i8 [%3], a1, b1, %6, T;\n"
            "tcgen05.mma.cta_group::2.kind::i8 [%3], a2, b2, %6, T;\n"
            "tcgen05.mma.cta_group::2.kind::i8 [%3], a3, b3, %6, T;\n"
            "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%9], both;\n"
            "selp.u32 %0, 1, 0, Q;\n"
            "}\n"
            : "=r"(ready)
            : "r"(next_full_bar), "r"(next_parity), "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate_first),
              "r"(sf), "r"(empty_bar), "r"(desc_hi)
            : "memory");
    }
    return ready;
}
// accumulator-complete signal to both CTAs of a pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile(
        "{\n.reg .b16 both;\nmov.b16 both, 3;\n"
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], both;\n}\n"
        ::"r"(bar) : "memory");
}

// TMA stage of one CTA of a pair: the loads land in this CTA's shared memory and report their bytes to the
// LEADER's full barrier (`leader_full_bar`, a shared::cluster address); only the leader announces the bytes
// (those of both CTAs).  No load is multicast.
__device__ __forceinline__ uint32_t tma_stage_2d_pair(uint32_t next_empty_bar, uint32_t next_parity, uint32_t leader_full_bar,
                                                      uint32_t tx_bytes_both, uint32_t is_leader, uint32_t dst_a,
                                                      const CUtensorMap *map_a, int32_t ax, int32_t ay, uint32_t dst_b,
                                                      const CUtensorMap *map_b, int32_t bx, int32_t by)
{
    uint32_t ready;
    asm volatile(
        "{\n"
        ".reg .pred Q, L;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 Q, [%1], %2;\n"
        "setp.ne.b32 L, %13, 0;\n"
        "@L mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%3], %4;\n"
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%5], [%6, {%7, %8}], [%3];\n"
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%9], [%10, {%11, %12}], [%3];\n"
        "selp.u32 %0, 1, 0, Q;\n"
        "}\n"
        : "=r"(ready)
        : "r"(next_empty_bar), "r"(next_parity), "r"(leader_full_bar), "r"(tx_bytes_both), "r"(dst_a), "l"(map_a), "r"(ax),
          "r"(ay), "r"(dst_b), "l"(map_b), "r"(bx), "r"(by), "r"(is_leader)
        : "memory");
    return ready;
}

// One pipeline stage of the TMA warp the same way: poll the NEXT stage's empty barrier first, announce this
// stage's bytes, issue its two loads, then read the poll's result.
__device__ __forceinline__ uint32_t tma_stage_2d(uint32_t next_empty_bar, uint32_t next_parity, uint32_t full_bar, uint32_t tx_bytes,
                                                 uint32_t dst_a, const CUtensorMap *map_a, int32_t ax, int32_t ay,
                                                 uint32_t dst_b, const CUtensorMap *map_b, int32_t bx, int32_t by)
{
    uint32_t ready;
    asm volatile(
        "{\n"
        ".reg .pred Q;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 Q, [%1], %2;\n"
        "mbarrier.arrive.expect_tx.shared::cta.b64 _, [%3], %4;\n"
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%5], [%6, {%7, %8}], [%3];\n"
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%9], [%10, {%11, %12}], [%3];\n"
        "selp.u32 %0, 1, 0, Q;\n"
        "}\n"
        : "=r"(ready)
        : "r"(next_empty_bar), "r"(next_parity), "r"(full_bar), "r"(tx_bytes), "r"(dst_a), "l"(map_a), "r"(ax), "r"(ay),
          "r"(dst_b), "l"(map_b), "r"(bx), "r"(by)
        : "memory");
    return ready;
}
__device__ __forceinline__ uint32_t tma_stage_conv(uint32_t next_empty_bar, uint32_t next_parity, uint32_t full_bar, uint32_t tx_bytes,
                                                   uint32_t dst_a, const CUtensorMap *map_a, int32_t c0, int32_t c1, int32_t c2,
                                                   int32_t c3, uint32_t dst_b, const CUtensorMap *map_b, int32_t bx, int32_t by)
{
    uint32_t ready;
    asm volatile(
        "{\n"
        ".reg .pred Q;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 Q, [%1], %2;\n"
        "mbarrier.arrive.expect_tx.shared::cta.b64 _, [%3], %4;\n"
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%5], [%6, {%7, %8, %9, %10}], [%3];\n"
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%11], [%12, {%13, %14}], [%3];\n"
        "selp.u32 %0, 1, 0, Q;\n"
        "}\n"
        : "=r"(ready)
        : "r"(next_empty_bar), "r"(next_parity), "r"(full_bar), "r"(tx_bytes), "r"(dst_a), "l"(map_a), "r"(c0), "r"(c1), "r"(c2),
          "r"(c3), "r"(dst_b), "l"(map_b), "r"(bx), "r"(by)
        : "memory");
    return ready;
}

// Diagnostic: one CTA waits, with a short limit, on a barrier that nothing ever arrives on.  No copy and no MMA is in
// flight, so the wait running out is all that happens: the status word is set through the same code path the product
// kernel's waits use, and the kernel returns.
constexpr int WAIT_PROBE_CODE = 9;
__global__ void __launch_bounds__(32) wait_probe_kernel()
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        (void)mbar_wait(smem_u32(&bar), 0, &abort_flag, WAIT_PROBE_CODE, 1u << 13);
    }
}

constexpr int next_pow2_cols(int c) { return c <= 32 ? 32 : c <= 64 ? 64 : c <= 128 ? 128 : c <= 256 ? 256 : 512; }

template <int FORM, int BN, int STG, int CTAS, int KB = BKB, int G = EPI_GROUPS>
struct TcCfg {
    static constexpr int A_BYTES = BM * KB;
    static constexpr int B_BYTES = (BN / CTAS) * KB;                    // a pair splits the B tile between its CTAs
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int CPW = (BN / 32 + G - 1) / G;                    // 32-column chunks per epilogue warp
    static constexpr int THR_WORDS = CPW * 32 + 8;                       // per epilogue warp: its thresholds + flip words
    static constexpr int THR_BYTES = 4 * G * THR_WORDS * 4;
    // epilogue staging per warp: one 4 KB tile of 32 x 32 int32 for the bulk stores; kernels instantiated
    // without it keep one more pipeline stage and store from registers
    static constexpr int STG_WARP_BYTES = STG ? 4096 : 0;
    static constexpr int STG_BYTES = 4 * G * STG_WARP_BYTES;
    static constexpr int AUX_BYTES = 256 + THR_BYTES + 1024;             // barriers, thresholds, 1024-byte alignment slack
    static constexpr int MAX_STAGES = (SMEM_LIMIT - AUX_BYTES - STG_BYTES) / STAGE_BYTES;
    static constexpr int STAGES = MAX_STAGES > 7 ? 7 : MAX_STAGES;
    static constexpr int SCALE_COL = 2 * BN;                             // FP4: unit block scales live behind the accumulators
    static constexpr int TMEM_COLS = next_pow2_cols(2 * BN + (FORM == QNN_FORM_FP4 ? 32 : 0));
    static constexpr int STG_OFFSET = STAGES * STAGE_BYTES;              // 1024-byte aligned like the stages
    static constexpr int BAR_OFFSET = STG_OFFSET + STG_BYTES;
    static constexpr int THR_OFFSET = BAR_OFFSET + 256;
    static constexpr int TOTAL = THR_OFFSET + THR_BYTES + 1024;
    static_assert(STAGES >= 3, "pipeline too shallow");
    static_assert(TMEM_COLS <= 512, "accumulators do not fit tensor memory");
    static_assert(BN % 32 == 0 && BN >= 32 && BN <= 256, "tile width");
    static_assert(CTAS == 1 || (CTAS == 2 && BN % 32 == 0), "pairs split B in two halves of whole 8-row groups");
    static_assert(KB == 128 || (KB == 64 && FORM == QNN_FORM_FP4 && CTAS == 1), "64-byte K blocks: e2m1, single CTA");
};

template <int FORM, int BN, int STG, int CTAS, int KB = BKB, int G = EPI_GROUPS>
__global__ void __launch_bounds__(tc_threads(G), 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               const __grid_constant__ CUtensorMap tmap_out, const TcParams p)
{
    using S = TcCfg<FORM, BN, STG, CTAS, KB, G>;
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
    // the next kernel in the stream may be scheduled as soon as SMs free up; it waits for this grid where it needs to
    griddep_launch_dependents();
    // In a pair (CTAS = 2) CTA 0 of the cluster leads: it owns the full and accumulator-empty barriers and issues
    // the MMAs; both CTAs load their halves of the operands and drain their 128 rows of the accumulator.
    const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;
    const bool leader = rank == 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4 * G * CTAS); }   // one arrival per epilogue warp
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc<CTAS>(smem_u32(tmem_slot), S::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync_all();                                 // the peer's barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (FORM == QNN_FORM_FP4) {
        // Unit scale factors (ue8m0 exponent 127 = 2^0) in 32 columns of every lane: whatever layout the
        // instruction reads its per-block scales in, every scale it finds is 1.0.
        if (warp >= 2 && warp < 6) {
            const int q = warp & 3;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                tmem_st8(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(S::SCALE_COL + 8 * c), 0x7f7f7f7fu);
            tmem_st_wait();
        }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }

    // Everything above (barriers, tensor memory, scales) touched only this CTA's own state and overlapped the tail of
    // the previous kernel; from here on global memory is read and written.
    griddep_wait();

    const uint32_t tiles_m = (uint32_t)p.tiles_m;                      // in units of BM * CTAS rows
    const uint32_t num_tiles = tiles_m * (uint32_t)p.tiles_n;          // below 2^31 (checked on the host)
    // a CTA, or a pair of them, walks the tiles blockIdx.x / CTAS, + gridDim.x / CTAS, ...  (written out in every
    // loop: held in named variables the two values cost the single-CTA kernel 12 % of its speed)

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            bool ready = false;                                    // this stage's slot is known to be free
            const uint32_t tx_bytes = ((uint32_t)p.a_tx_bytes + (uint32_t)S::B_BYTES) * CTAS;   // the leader announces both CTAs' bytes
            // destination, barriers and the K coordinate are carried from stage to stage (see the MMA warp)
            const uint32_t fb0 = (CTAS == 2) ? map_to_cta(full_bar(0), 0) : full_bar(0), eb0 = empty_bar(0);
            uint32_t sa = base, fb = fb0, eb = eb0;
            // tile coordinates advance by additions: one division per role, before its loop
            const uint32_t step_n = (gridDim.x / CTAS) / tiles_m, step_m = (gridDim.x / CTAS) - step_n * tiles_m;
            int32_t tn = (int32_t)((blockIdx.x / CTAS) / tiles_m), tm = (int32_t)((blockIdx.x / CTAS) - (uint32_t)tn * tiles_m);
            for (uint32_t t = blockIdx.x / CTAS; t < num_tiles && ok; t += gridDim.x / CTAS) {
                int32_t img = 0, y0 = 0;
                if (p.conv) { img = tm / p.tiles_per_img; y0 = (tm - img * p.tiles_per_img) * p.cR; img *= p.cG; }
                int32_t cx = 0, kx = 0, tx = -p.cpad, ty = y0 - p.cpad;   // conv: channel byte, K byte, tap column and row of kb
                const int32_t a_row = (CTAS == 2) ? (tm * 2 + (int32_t)rank) * BM : tm * BM;
                const int32_t b_row = (CTAS == 2) ? tn * BN + (int32_t)rank * ((tn == p.tiles_n - 1 ? p.n_last : BN) / 2) : tn * BN;
                const int32_t cx_end = p.cblocks * KB, tx_end = p.cKW - p.cpad;
                // (the convolution's loop is unrolled, the plain one is not: measured best for each)
                if (p.conv) {
#pragma unroll 4
                    for (int32_t kb = 0; kb < p.num_kb; ++kb) {
                        if (!ready && !mbar_wait(eb, phase ^ 1u, abort_flag, 1)) { ok = false; break; }
                        const bool wrap = stage == S::STAGES - 1;
                        const uint32_t sa_n = wrap ? base : sa + (uint32_t)S::STAGE_BYTES;
                        const uint32_t fb_n = wrap ? fb0 : fb + 8u;
                        const uint32_t eb_n = wrap ? eb0 : eb + 8u;
                        const uint32_t phase_n = wrap ? phase ^ 1u : phase;
                        ready = tma_stage_conv(eb_n, phase_n ^ 1u, fb, tx_bytes, sa, &tmap_a, cx, tx, ty, img, sa + S::A_BYTES, &tmap_b, kx,
                                               b_row) != 0;
                        cx += KB; kx += KB;
                        if (cx == cx_end) { cx = 0; if (++tx == tx_end) { tx = -p.cpad; ++ty; } }
                        stage = wrap ? 0 : stage + 1;
                        sa = sa_n; fb = fb_n; eb = eb_n; phase = phase_n;
                    }
                } else {
#pragma unroll 1
                    for (int32_t kb = 0; kb < p.num_kb; ++kb) {
                        if (!ready && !mbar_wait(eb, phase ^ 1u, abort_flag, 1)) { ok = false; break; }
                        const bool wrap = stage == S::STAGES - 1;
                        const uint32_t sa_n = wrap ? base : sa + (uint32_t)S::STAGE_BYTES;
                        const uint32_t fb_n = wrap ? fb0 : fb + 8u;
                        const uint32_t eb_n = wrap ? eb0 : eb + 8u;
                        const uint32_t phase_n = wrap ? phase ^ 1u : phase;
                        if (CTAS == 2)
                            ready = tma_stage_2d_pair(eb_n, phase_n ^ 1u, fb, tx_bytes, (uint32_t)leader, sa, &tmap_a, kx, a_row,
                                                      sa + S::A_BYTES, &tmap_b, kx, b_row) != 0;
                        else
                            ready = tma_stage_2d(eb_n, phase_n ^ 1u, fb, tx_bytes, sa, &tmap_a, kx, a_row, sa + S::A_BYTES, &tmap_b, kx,
                                                 b_row) != 0;
                        kx += KB;
                        stage = wrap ? 0 : stage + 1;
                        sa = sa_n; fb = fb_n; eb = eb_n; phase = phase_n;
                    }
                }
                tm += (int32_t)step_m; tn += (int32_t)step_n;
                if (tm >= (int32_t)tiles_m) { tm -= (int32_t)tiles_m; ++tn; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            int stage = 0; uint32_t phase = 0;
            uint32_t iter = 0;
            bool ok = true;
            bool ready = false;                                    // this stage's operands are known to have landed
            const uint32_t sf = tmem_base + (uint32_t)S::SCALE_COL;
            // A stage's descriptors differ only in the address field of their low words, and everything a K step needs
            // (descriptor words, barrier addresses) is carried from stage to stage by one addition or a wrap-around:
            // the issuing thread runs one dependent instruction every few clocks, so every instruction here counts.
            const uint64_t desc0 = make_kmajor_desc<KB>(base);
            const uint32_t desc_hi = (uint32_t)(desc0 >> 32);
            const uint32_t a_lo0 = (uint32_t)desc0, fb0 = full_bar(0), eb0 = empty_bar(0);
            uint32_t a_lo = a_lo0, fb = fb0, eb = eb0;
            const uint32_t step_n = (gridDim.x / CTAS) / tiles_m, step_m = (gridDim.x / CTAS) - step_n * tiles_m;
            uint32_t tn = (blockIdx.x / CTAS) / tiles_m, tm = (blockIdx.x / CTAS) - tn * tiles_m;
            for (uint32_t t = blockIdx.x / CTAS; t < num_tiles && ok; t += gridDim.x / CTAS, ++iter) {
                const uint32_t as = iter & 1u, aphase = (iter >> 1) & 1u;
                const uint32_t idesc = (tn == (uint32_t)p.tiles_n - 1u) ? p.idesc_last : p.idesc;
                tm += step_m; tn += step_n;
                if (tm >= tiles_m) { tm -= tiles_m; ++tn; }
                if (!mbar_wait(tempty_bar(as), aphase ^ 1u, abort_flag, 2)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + as * (uint32_t)BN;
                // (unrolled by four: measured 9 % faster on the 10000 x 4096 x 4096 product than not unrolled; by 3, 6 or 8 is slower)
#pragma unroll 4
                for (int32_t kb = 0; kb < p.num_kb; ++kb) {
                    if (!ready && !mbar_wait(fb, phase, abort_flag, 3)) { ok = false; break; }
                    const bool wrap = stage == S::STAGES - 1;
                    const uint32_t a_lo_n = wrap ? a_lo0 : a_lo + (uint32_t)(S::STAGE_BYTES >> 4);
                    const uint32_t fb_n = wrap ? fb0 : fb + 8u;
                    const uint32_t eb_n = wrap ? eb0 : eb + 8u;
                    const uint32_t phase_n = wrap ? phase ^ 1u : phase;
                    const uint32_t b_lo = a_lo + (uint32_t)(S::A_BYTES >> 4);
                    if (CTAS == 2)
                        ready = umma_stage_pair<FORM>(fb_n, phase_n, d_tmem, a_lo, b_lo, desc_hi, idesc, (uint32_t)(kb != 0), sf, eb) != 0;
                    else if (KB == 64)
                        ready = umma_stage_half(fb_n, phase_n, d_tmem, a_lo, b_lo, desc_hi, idesc, (uint32_t)(kb != 0), sf, eb) != 0;
                    else
                        ready = umma_stage<FORM>(fb_n, phase_n, d_tmem, a_lo, b_lo, desc_hi, idesc, (uint32_t)(kb != 0), sf, eb) != 0;
                    stage = wrap ? 0 : stage + 1;
                    a_lo = a_lo_n; fb = fb_n; eb = eb_n; phase = phase_n;
                }
                if (ok) {                                        // accumulator complete
                    if (CTAS == 2) umma_commit_pair(tfull_bar(as));
                    else umma_commit(tfull_bar(as));
                }
            }
        }
    } else {
        // EPI_GROUPS warps share each quarter of the accumulator's lanes; group g drains the 32-column chunks
        // g, g + EPI_GROUPS, ...  One warp alone on a scheduler cannot hide the latency of its own dependent
        // instructions, so the epilogue's time per tile falls almost linearly with the number of groups.
        const int q = warp & 3;                                  // TMEM lane quarter this warp may read
        const int grp = (warp - 2) >> 2;                         // which chunks of the tile it drains
        const int ew = grp * 4 + q;
        constexpr int CPW = S::CPW;                              // chunks per warp
        int32_t *thr_w = reinterpret_cast<int32_t *>(gen + S::THR_OFFSET) + ew * S::THR_WORDS;  // this warp's thresholds
        uint32_t *flip_w = reinterpret_cast<uint32_t *>(thr_w + CPW * 32);                      // and flip words
        uint8_t *stg = gen + S::STG_OFFSET + ew * S::STG_WARP_BYTES;                            // this warp's staging tile
        const uint32_t stg_u32 = base + (uint32_t)(S::STG_OFFSET + ew * S::STG_WARP_BYTES);
        const bool want_bits = p.out_bits != nullptr;
        const bool want_form = p.out_form != nullptr;
        const bool want_sign = want_bits || want_form;
        const bool form_fp4 = p.out_form_kind == QNN_FORM_FP4;
        uint32_t iter = 0;
        bool ok = true;
        // lane l holds the thresholds of columns c*32 + l of this warp's chunks c = grp + lc*EPI_GROUPS and, as bit lc,
        // their flips
        int32_t thr_next[CPW];
        uint8_t flip_raw[CPW];
        auto fetch_thresholds = [&](int64_t ncol0) {
#pragma unroll
            for (int lc = 0; lc < CPW; ++lc) {
                const int64_t n = ncol0 + (grp + lc * G) * 32 + lane;
                const bool ncol = (grp + lc * G) < BN / 32 && n < p.N;
                // (raw values: nothing here may wait for the loads -- they are converted when they are parked)
                const int32_t tv = ncol ? __ldg(p.thr + n) : 0;
                thr_next[lc] = tv;
                if (ncol && p.flip) flip_raw[lc] = __ldg(p.flip + n);
                else flip_raw[lc] = 0;
            }
        };
        // Consecutive tiles of a CTA mostly share their column block, so thresholds are fetched and parked only when
        // the column block changes: tn_fetched is the block whose values the registers hold, tn_parked the one in
        // shared memory.
        int32_t tn_fetched = -1, tn_parked = -1;
        // convolution: where this thread's row sits inside a tile never changes (image of the tile, row, column)
        int32_t r_gi = 0, r_y = 0, r_x = 0;
        if (p.conv) {
            const int32_t r = q * 32 + lane;
            r_gi = r / (p.cR * p.cW);
            const int32_t rem = r - r_gi * (p.cR * p.cW);
            r_y = rem / p.cW;
            r_x = rem - r_y * p.cW;
        }
        const uint32_t step_n = (gridDim.x / CTAS) / tiles_m, step_m = (gridDim.x / CTAS) - step_n * tiles_m;
        int32_t tn = (int32_t)((blockIdx.x / CTAS) / tiles_m), tm = (int32_t)((blockIdx.x / CTAS) - (uint32_t)tn * tiles_m);
        if (want_sign && blockIdx.x / CTAS < num_tiles) {
            tn_fetched = tn;
            fetch_thresholds((int64_t)tn_fetched * BN);
        }
        for (uint32_t t = blockIdx.x / CTAS; t < num_tiles && ok; t += gridDim.x / CTAS, ++iter) {
            // the next tile's coordinates
            int32_t tm_next = tm + (int32_t)step_m, tn_next = tn + (int32_t)step_n;
            if (tm_next >= (int32_t)tiles_m) { tm_next -= (int32_t)tiles_m; ++tn_next; }
            const uint32_t as = iter & 1u, aphase = (iter >> 1) & 1u;
            const int64_t ntile = (int64_t)tn * BN;

            // Thresholds and flip bytes of this tile's column block were fetched into registers a tile ago (or just
            // before the loop): park them in this warp's shared rows, then start fetching the next block's, so that
            // their global-memory latency never sits between two tiles.
            if (want_sign && tn != tn_parked) {                  // (warp-uniform)
                tn_parked = tn;
                __syncwarp();
#pragma unroll
                for (int lc = 0; lc < CPW; ++lc) {
                    int32_t tv = thr_next[lc];
                    if (FORM == QNN_FORM_FP4) {
                        // accumulators are exact integers below 2^24 held as floats: compare there.  A threshold
                        // beyond +-2^24 decides the same way as +-2^24, which a float holds exactly.
                        tv = tv > (1 << 24) ? (1 << 24) : (tv < -(1 << 24) ? -(1 << 24) : tv);
                        // (a zero threshold is parked as -0.0: a sum that came out as -0.0 then gives -0.0 - (-0.0) = +0.0,
                        // whose clear sign bit is the right answer to 0 >= 0; +0.0 would give -0.0)
                        tv = tv == 0 ? (int32_t)0x80000000u : __float_as_int((float)tv);
                    } else if (p.thr_clamp > 0) {
                        // |sum| <= thr_clamp - 1 < 2^30: a threshold beyond +-thr_clamp decides like +-thr_clamp, and
                        // sum - threshold then cannot overflow, so its sign bit is the comparison
                        tv = tv > p.thr_clamp ? p.thr_clamp : (tv < -p.thr_clamp ? -p.thr_clamp : tv);
                    }
                    thr_w[lc * 32 + lane] = tv;
                    const uint32_t fw = __ballot_sync(0xffffffffu, flip_raw[lc] != 0);
                    if (lane == lc) flip_w[lc] = fw;
                }
                __syncwarp();
            }
            if (want_sign) {
                const uint32_t tnext = t + gridDim.x / CTAS;
                if (tnext < num_tiles) {
                    if (tn_next != tn_fetched) { tn_fetched = tn_next; fetch_thresholds((int64_t)tn_next * BN); }
                }
            }

            // which output row this thread owns
            const int r = q * 32 + lane;
            int64_t m, m_warp0;                                  // this thread's row, and the row of the warp's lane 0
            bool mrow;
            int64_t m_st = 0;                                    // row and predicate of the sign outputs (differ when pooling)
            bool st_ok = false;
            int32_t cls = 0, c_img = 0, c_pix0 = 0;
            if (p.conv) {
                // a tile is cR rows of one image, or cG whole images one after the other
                const int32_t tile_img = tm / p.tiles_per_img;
                const int32_t y0 = (tm - tile_img * p.tiles_per_img) * p.cR;
                const int32_t gi = r_gi;
                const int32_t y = y0 + r_y;
                const int32_t x = r_x;
                c_img = tile_img * p.cG + gi;
                mrow = (gi < p.cG) && (y < p.cH) && (c_img < p.cB);
                m = ((int64_t)c_img * p.cH + y) * p.cW + x;
                c_pix0 = y0 * p.cW + q * 32;
                m_warp0 = (int64_t)tile_img * p.cG * p.cH * p.cW + c_pix0;
                if (p.pool) {
                    // the even-row, even-column pixel of every 2 x 2 window writes the pooled pixel
                    st_ok = mrow && ((x & 1) == 0) && ((y & 1) == 0);
                    m_st = ((int64_t)c_img * (p.cH >> 1) + (y >> 1)) * (p.cW >> 1) + (x >> 1);
                }
                const int32_t pd = p.cpad, pc = pd + 1;
                const int32_t ty = max(pd - y, 0), by = max(y + pd - (p.cH - 1), 0);
                const int32_t tx = max(pd - x, 0), bx = max(x + pd - (p.cW - 1), 0);
                cls = mrow ? ((ty * pc + by) * pc + tx) * pc + bx : 0;
            } else {
                m = ((int64_t)tm * CTAS + rank) * BM + r;
                m_warp0 = ((int64_t)tm * CTAS + rank) * BM + q * 32;
                mrow = m < p.M;
            }
            if (!p.pool) { m_st = m; st_ok = mrow; }
            const bool any_border = p.conv ? (__any_sync(0xffffffffu, cls != 0) != 0) : false;
            int64_t img = 0, pix = 0;                            // where an int32 NCHW result of this row goes
            if (p.epilogue == EPI_NCHW && mrow && p.out != nullptr) {
                if (p.conv) { img = c_img; pix = m - (int64_t)c_img * p.cH * p.cW; }
                else { img = m / p.hw; pix = m - img * p.hw; }
            }

            // the tensor-memory loads below are warp-collective: leave the loop only as a whole warp
            if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(as), aphase, abort_flag, 4))) { ok = false; break; }
            tc_fence_after();

            // this warp's share of the accumulator, 32 columns at a time
            const uint32_t tacc = tmem_base + ((uint32_t)(q * 32) << 16) + as * (uint32_t)BN;
            int nchunks = (int)((p.N - ntile + 31) >> 5);         // warp-uniform
            nchunks = nchunks > BN / 32 ? BN / 32 : nchunks;
#pragma unroll 1
            for (int c = grp, lc = 0; c < nchunks; c += G, ++lc) {
                const int64_t n0 = ntile + c * 32;
                uint32_t v[32];
                tmem_ld32(tacc + (uint32_t)(c * 32), v);
                // Border corrections.  e2m1: the fp32 accumulators are exact integers, so the correction is added in float.
                if (any_border) {
                    // every lane adds the row of its own class (class 0, the interior, is a row of zeros): eight
                    // independent loads, lanes of one class sharing their addresses
                    const int4 *cp = reinterpret_cast<const int4 *>(p.corr + (int64_t)cls * p.corr_ld + n0);
                    int4 cv[8];
#pragma unroll
                    for (int j4 = 0; j4 < 8; ++j4) cv[j4] = __ldg(cp + j4);
#pragma unroll
                    for (int j4 = 0; j4 < 8; ++j4) {
                        if (FORM == QNN_FORM_FP4) {
                            v[4 * j4] = __float_as_uint(__uint_as_float(v[4 * j4]) + (float)cv[j4].x);
                            v[4 * j4 + 1] = __float_as_uint(__uint_as_float(v[4 * j4 + 1]) + (float)cv[j4].y);
                            v[4 * j4 + 2] = __float_as_uint(__uint_as_float(v[4 * j4 + 2]) + (float)cv[j4].z);
                            v[4 * j4 + 3] = __float_as_uint(__uint_as_float(v[4 * j4 + 3]) + (float)cv[j4].w);
                        } else {
                            v[4 * j4] += (uint32_t)cv[j4].x; v[4 * j4 + 1] += (uint32_t)cv[j4].y;
                            v[4 * j4 + 2] += (uint32_t)cv[j4].z; v[4 * j4 + 3] += (uint32_t)cv[j4].w;
                        }
                    }
                }
                int32_t iv[32];
                if (FORM != QNN_FORM_FP4 || p.out != nullptr) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        iv[j] = (FORM == QNN_FORM_FP4) ? __float2int_rn(__uint_as_float(v[j])) : (int32_t)v[j];
                }
                if (p.out != nullptr) {
                    if (STG && p.tma_out) {
                        // registers -> staging tile -> one asynchronous bulk store per 32 x 32 block
                        uint8_t *buf = stg;
                        if (lane == 0) bulk_wait_read<0>();      // this warp's previous store has read the tile
                        __syncwarp();
                        if (p.tma_out == 1) {
                            // [row][32 columns], 16-byte chunks swizzled by the row (the tensor map's 128-byte swizzle)
#pragma unroll
                            for (int ch = 0; ch < 8; ++ch)
                                *reinterpret_cast<int4 *>(buf + lane * 128 + ((ch ^ (lane & 7)) << 4)) =
                                    make_int4(iv[4 * ch], iv[4 * ch + 1], iv[4 * ch + 2], iv[4 * ch + 3]);
                        } else {
                            // [channel][32 pixels]: a row of 32 lanes is one 128-byte line
#pragma unroll
                            for (int j = 0; j < 32; ++j) *reinterpret_cast<int32_t *>(buf + j * 128 + lane * 4) = iv[j];
                        }
                        fence_async_shared();
                        __syncwarp();
                        if (lane == 0) {
                            if (p.tma_out == 1) tma_store_2d(&tmap_out, (int32_t)n0, (int32_t)m_warp0, stg_u32);
                            else tma_store_3d(&tmap_out, c_pix0, (int32_t)n0, c_img, stg_u32);
                            bulk_commit();
                        }
                    } else if (mrow) {
                        if (p.epilogue == EPI_NCHW) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (n0 + j < p.N) p.out[(img * p.N + n0 + j) * p.hw + pix] = iv[j];
                        } else {
                            int32_t *dst = p.out + m * p.ldo + n0;
                            if (n0 + 32 <= p.N && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0)) {
#pragma unroll
                                for (int j = 0; j < 32; j += 4)
                                    *reinterpret_cast<int4 *>(dst + j) = make_int4(iv[j], iv[j + 1], iv[j + 2], iv[j + 3]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (n0 + j < p.N) dst[j] = iv[j];
                            }
                        }
                    }
                }
                if (want_sign) {
                    const int4 *t4 = reinterpret_cast<const int4 *>(thr_w + lc * 32);
                    uint32_t w = 0;
                    if (FORM == QNN_FORM_FP4 || p.thr_clamp > 0) {
                        // bit j = (acc_j >= thr_j) = NOT sign(acc_j - thr_j): one subtraction and one funnel shift per
                        // column (e2m1: in float, exact; int8: no overflow after the clamp), last column first so that
                        // column 0 lands in bit 0; four independent byte-wide chains keep the shifts from serialising
                        uint32_t wb[4];
#pragma unroll
                        for (int g4 = 0; g4 < 4; ++g4) {
                            uint32_t x = 0;
#pragma unroll
                            for (int h = 1; h >= 0; --h) {
                                const int4 tt = t4[2 * g4 + h];  // same address in every lane: a broadcast read
                                const int j = 8 * g4 + 4 * h;
                                if (FORM == QNN_FORM_FP4) {
                                    x = __funnelshift_l(__float_as_uint(__uint_as_float(v[j + 3]) - __int_as_float(tt.w)), x, 1);
                                    x = __funnelshift_l(__float_as_uint(__uint_as_float(v[j + 2]) - __int_as_float(tt.z)), x, 1);
                                    x = __funnelshift_l(__float_as_uint(__uint_as_float(v[j + 1]) - __int_as_float(tt.y)), x, 1);
                                    x = __funnelshift_l(__float_as_uint(__uint_as_float(v[j]) - __int_as_float(tt.x)), x, 1);
                                } else {
                                    x = __funnelshift_l((uint32_t)(iv[j + 3] - tt.w), x, 1);
                                    x = __funnelshift_l((uint32_t)(iv[j + 2] - tt.z), x, 1);
                                    x = __funnelshift_l((uint32_t)(iv[j + 1] - tt.y), x, 1);
                                    x = __funnelshift_l((uint32_t)(iv[j] - tt.x), x, 1);
                                }
                            }
                            wb[g4] = x;
                        }
                        w = ~(wb[0] | (wb[1] << 8) | (wb[2] << 16) | (wb[3] << 24));
                    } else {
#pragma unroll
                        for (int j4 = 0; j4 < 8; ++j4) {
                            const int4 tt = t4[j4];
                            w |= (uint32_t)(iv[4 * j4] >= tt.x) << (4 * j4);
                            w |= (uint32_t)(iv[4 * j4 + 1] >= tt.y) << (4 * j4 + 1);
                            w |= (uint32_t)(iv[4 * j4 + 2] >= tt.z) << (4 * j4 + 2);
                            w |= (uint32_t)(iv[4 * j4 + 3] >= tt.w) << (4 * j4 + 3);
                        }
                    }
                    const int64_t left = p.N - n0;
                    const uint32_t nmask = left >= 32 ? 0xffffffffu : ((1u << (int)left) - 1u);
                    w = (w ^ flip_w[lc]) & nmask;
                    if (p.pool) {
                        // Max-pooling sits between the convolution and the threshold (Table 7); the threshold is monotone
                        // in the sum, so the pooled sign is the OR of the window's four signs, the AND where the
                        // comparison is flipped.  The window's pixels are lanes l, l^1 (next column), l^W, l^W^1 (next row).
                        const uint32_t f = flip_w[lc];
                        uint32_t wo = w, wa = w;
                        wo |= __shfl_xor_sync(0xffffffffu, wo, 1);
                        wa &= __shfl_xor_sync(0xffffffffu, wa, 1);
                        wo |= __shfl_xor_sync(0xffffffffu, wo, p.cW);
                        wa &= __shfl_xor_sync(0xffffffffu, wa, p.cW);
                        w = ((wo & ~f) | (wa & f)) & nmask;
                    }
                    if (want_bits && st_ok) p.out_bits[m_st * p.ld_bits + (n0 >> 5)] = w;
                    if (want_form) {
                        if (form_fp4) {
                            // +1 -> e2m1 0x2, -1 -> 0xA, columns past N -> 0
                            uint32_t o[4];
#pragma unroll
                            for (int b = 0; b < 4; ++b) o[b] = 0xAAAAAAAAu ^ (spread_bits_to_nibbles((w >> (8 * b)) & 0xffu) << 3);
                            if (left < 32) {                     // warp-uniform: only the last chunk of a ragged N
#pragma unroll
                                for (int b = 0; b < 4; ++b) o[b] &= spread_bits_to_nibbles((nmask >> (8 * b)) & 0xffu) * 0xfu;
                            }
                            const uint4 o4 = make_uint4(o[0], o[1], o[2], o[3]);
                            if (st_ok) *reinterpret_cast<uint4 *>(p.out_form + m_st * p.ld_form + (n0 >> 1)) = o4;
                        } else {
                            // +1 -> 0x01, -1 -> 0xFF, columns past N -> 0
                            uint32_t o[8];
#pragma unroll
                            for (int b = 0; b < 8; ++b) {
                                const uint32_t sb = spread_bits_to_bytes((w >> (4 * b)) & 0xfu);
                                const uint32_t vm = spread_bits_to_bytes((nmask >> (4 * b)) & 0xfu) * 0xffu;
                                o[b] = (0xFFFFFFFFu ^ (sb * 0xfeu)) & vm;
                            }
                            uint4 *dst = reinterpret_cast<uint4 *>(p.out_form + m_st * p.ld_form + n0);
                            if (st_ok) {
                                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
                            }
                        }
                    }
                }
            }
            // all TMEM reads of this accumulator stage are done: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CTAS == 2) mbar_arrive_cluster(map_to_cta(tempty_bar(as), 0));
                else mbar_arrive(tempty_bar(as));
            }
            tm = tm_next; tn = tn_next;
        }
        // stores still reading shared memory must finish before the block's shared memory goes away
        if (STG) {
            if (lane == 0) bulk_wait_all();
            __syncwarp();
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
    if (CTAS == 2) cluster_sync_all();     // the peer no longer touches this CTA's barriers, shared or tensor memory
    tc_fence_after();
    if (warp == 1) tmem_dealloc<CTAS>(tmem_base, S::TMEM_COLS);
}

// ---- expansion of packed planes to tensor-core forms ---------------------------
//
// `period`/`tail` say where pad bits sit: word (w mod period) == period-1 has only `tail` valid
// bits; every pad position expands to the value 0.

// int8 form: one thread produces 16 consecutive bytes (half a source word) of a row.  IDX is the index type:
// 32-bit arithmetic whenever the element count allows it (the 64-bit divisions would dominate the kernel).
template <typename IDX>
__global__ void __launch_bounds__(256) expand_i8_kernel(const uint32_t *__restrict__ planes, int nplanes, int pm1,
                                                        int64_t ld, int64_t plane_stride, int64_t rows, int64_t kwords,
                                                        int64_t period64, int tail, uint8_t *__restrict__ out, int64_t out_ld)
{
    griddep_launch_dependents();
    griddep_wait();
    const IDX chunks = (IDX)(kwords * 2);
    const IDX total = (IDX)rows * chunks;
    const IDX period = (IDX)period64;
    const uint32_t lcode = (1u << nplanes) - 1u;
    for (IDX e = (IDX)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (IDX)gridDim.x * blockDim.x) {
        const IDX r = e / chunks;
        const IDX ch = e - r * chunks;
        const IDX widx = ch >> 1;
        const int half = (int)(ch & 1);
        const bool ragged = tail < 32 && ((widx % period) == period - 1);      // this word holds pad bits
        uint32_t acc[4] = {0u, 0u, 0u, 0u};
        for (int i = 0; i < nplanes; ++i) {
            const uint32_t w = __ldg(planes + i * plane_stride + (int64_t)r * ld + widx);
            const uint32_t h = (w >> (16 * half)) & 0xffffu;
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) acc[nb] += spread_bits_to_bytes((h >> (4 * nb)) & 0xfu) << i;
        }
        uint32_t o[4];
#pragma unroll
        for (int nb = 0; nb < 4; ++nb) {
            uint32_t v = acc[nb];
            if (pm1) v = __vsub4(v << 1, lcode * 0x01010101u);                  // 2q - (2^k - 1) per byte
            o[nb] = v;
        }
        if (ragged) {
            const uint32_t vm = (((1u << tail) - 1u) >> (16 * half)) & 0xffffu;
#pragma unroll
            for (int nb = 0; nb < 4; ++nb) o[nb] &= spread_bits_to_bytes((vm >> (4 * nb)) & 0xfu) * 0xffu;
        }
        *reinterpret_cast<uint4 *>(out + (int64_t)r * out_ld + (int64_t)ch * 16) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// e2m1 code of an integer value in {0, +-1, +-2, +-3}: sign bit 3; magnitudes 1 -> 0b010, 2 -> 0b100, 3 -> 0b101.
// fp4 form: one thread turns one source word (per plane) into 32 nibbles = 16 bytes.
template <typename IDX>
__global__ void __launch_bounds__(256) expand_fp4_kernel(const uint32_t *__restrict__ planes, int nplanes, int pm1,
                                                         int64_t ld, int64_t plane_stride, int64_t rows, int64_t kwords64,
                                                         int64_t period64, int tail, uint8_t *__restrict__ out, int64_t out_ld)
{
    griddep_launch_dependents();
    griddep_wait();
    const IDX kwords = (IDX)kwords64;
    const IDX total = (IDX)rows * kwords;
    const IDX period = (IDX)period64;
    for (IDX e = (IDX)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (IDX)gridDim.x * blockDim.x) {
        const IDX r = e / kwords;
        const IDX w = e - r * kwords;
        const bool ragged = tail < 32 && ((w % period) == period - 1);         // this word holds pad bits
        const uint32_t p0 = __ldg(planes + (int64_t)r * ld + w);
        const uint32_t p1 = nplanes > 1 ? __ldg(planes + plane_stride + (int64_t)r * ld + w) : 0u;
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
                    const uint32_t neg = (s1 ^ 0x11111111u) << 3;               // sign: negative while plane 1 is clear
                    const uint32_t three = ~(s0 ^ s1) & 0x11111111u;            // |value| = 3 when both planes agree
                    code = neg | (three * 0x5u) | ((three ^ 0x11111111u) << 1);  // 3 -> 0b101, 1 -> 0b010
                }
            } else {
                // unsigned code q = s0 + 2*s1: 0 -> 0, 1 -> 0b010, 2 -> 0b100, 3 -> 0b101
                const uint32_t s1 = spread_bits_to_nibbles((p1 >> (8 * b)) & 0xffu);
                code = (s1 << 2) | ((s0 & ~s1) << 1) | (s0 & s1);
            }
            o[b] = code;
        }
        if (ragged) {
            const uint32_t vword = (1u << tail) - 1u;
#pragma unroll
            for (int b = 0; b < 4; ++b) o[b] &= spread_bits_to_nibbles((vword >> (8 * b)) & 0xffu) * 0xfu;
        }
        *reinterpret_cast<uint4 *>(out + (int64_t)r * out_ld + (int64_t)w * 16) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// ---- tensor maps -------------------------------------------------------------

// 2-D byte matrix [rows, row_bytes] with rows ld_bytes apart; box = 128 bytes x box_rows; reads past either extent give 0
int make_map_2d(CUtensorMap *map, const void *base, int64_t rows, int64_t row_bytes, int64_t ld_bytes, int box_rows, int kblk = BKB)
{
    EncodeTiledFn fn = encode_fn();
    QNN_REQUIRE(fn != nullptr, QNN_ERR_CUDA, "tc gemm: cuTensorMapEncodeTiled is not available from this driver");
    cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld_bytes};
    cuuint32_t box[2] = {(cuuint32_t)kblk, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, kblk == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    QNN_REQUIRE(r == CUDA_SUCCESS, QNN_ERR_CUDA, "tc gemm: cuTensorMapEncodeTiled failed with code %d", (int)r);
    return QNN_OK;
}

// 4-D NHWC byte tensor [B, H, W, cbytes]; box = 128 bytes x W x box_h x 1
int make_map_nhwc(CUtensorMap *map, const void *base, int B, int H, int W, int64_t cbytes, int box_h, int box_b, int kblk)
{
    EncodeTiledFn fn = encode_fn();
    QNN_REQUIRE(fn != nullptr, QNN_ERR_CUDA, "tc conv: cuTensorMapEncodeTiled is not available from this driver");
    cuuint64_t dims[4] = {(cuuint64_t)cbytes, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)cbytes, (cuuint64_t)cbytes * W, (cuuint64_t)cbytes * W * H};
    cuuint32_t box[4] = {(cuuint32_t)kblk, (cuuint32_t)W, (cuuint32_t)box_h, (cuuint32_t)box_b};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, kblk == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    QNN_REQUIRE(r == CUDA_SUCCESS, QNN_ERR_CUDA, "tc conv: cuTensorMapEncodeTiled failed with code %d", (int)r);
    return QNN_OK;
}

// destination maps of the epilogue's bulk stores
int make_map_out(CUtensorMap *map, CUtensorMapDataType type, int rank, void *base, const cuuint64_t *dims,
                 const cuuint64_t *strides, const cuuint32_t *box, CUtensorMapSwizzle swz)
{
    EncodeTiledFn fn = encode_fn();
    QNN_REQUIRE(fn != nullptr, QNN_ERR_CUDA, "tc gemm: cuTensorMapEncodeTiled is not available from this driver");
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, type, (cuuint32_t)rank, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                    CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    QNN_REQUIRE(r == CUDA_SUCCESS, QNN_ERR_CUDA, "tc gemm: cuTensorMapEncodeTiled (output) failed with code %d", (int)r);
    return QNN_OK;
}

// CTA pairs a persistent grid of this kernel can keep resident at once (0 = pairs cannot be launched)
template <int FORM, int BN, int STG>
int max_pairs()
{
    using S = TcCfg<FORM, BN, STG, 2>;
    auto kern = gemm_tc_kernel<FORM, BN, STG, 2>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL) != cudaSuccess) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)sm_count());
    cfg.blockDim = dim3(TC_THREADS);
    cfg.dynamicSmemBytes = S::TOTAL;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    return n;
}

// The same, asked once per device ordinal (the answer depends on the device's SM count and shared memory) and kept;
// two host threads racing on the first call compute the same number.
int pairs_resident_on_current_device()
{
    static std::atomic<int> cached[64];                 // 0 = not asked yet; stored as pairs + 1
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    int v = cached[dev].load(std::memory_order_acquire);
    if (v == 0) {
        v = max_pairs<QNN_FORM_FP4, 224, 0>() + 1;
        cached[dev].store(v, std::memory_order_release);
    }
    return v - 1;
}

template <int FORM, int BN, int STG, int CTAS, int KB = BKB, int G = EPI_GROUPS>
int launch_tc_stg(const CUtensorMap &ma, const CUtensorMap &mb, const CUtensorMap &mo, TcParams p, int workers, cudaStream_t st)
{
    using S = TcCfg<FORM, BN, STG, CTAS, KB, G>;
    auto kern = gemm_tc_kernel<FORM, BN, STG, CTAS, KB, G>;
    // the shared-memory opt-in is per kernel and device: asked for once, not on every launch (it costs microseconds)
    // (per device ordinal; racing first calls of two host threads both set the same attribute, which is harmless)
    static std::atomic<bool> opted_in[64];
    int dev = 0;
    QNN_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64 || !opted_in[dev].load(std::memory_order_acquire)) {
        QNN_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::TOTAL));
        if (dev >= 0 && dev < 64) opted_in[dev].store(true, std::memory_order_release);
    }
    const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n;
    QNN_REQUIRE(tiles < ((int64_t)1 << 31), QNN_ERR_UNSUPPORTED, "tc gemm: too many output tiles");
    const int nw = (int)(tiles < workers ? tiles : workers);
    profile_before(st);
    {
        // programmatic stream serialisation: the grid may be scheduled while the previous kernel drains (the kernel
        // calls griddepcontrol.wait before it touches global memory); QNN_PDL=0 in the environment turns it off
        const bool pdl = pdl_enabled();
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(CTAS * nw));
        cfg.blockDim = dim3(tc_threads(G));
        cfg.dynamicSmemBytes = S::TOTAL;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        unsigned na = 0;
        if (CTAS == 2) {
            attr[na].id = cudaLaunchAttributeClusterDimension;
            attr[na].val.clusterDim.x = 2; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
            ++na;
        }
        if (pdl) {
            attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[na].val.programmaticStreamSerializationAllowed = 1;
            ++na;
        }
        cfg.attrs = attr; cfg.numAttrs = na;
        QNN_CUDA(cudaLaunchKernelEx(&cfg, kern, ma, mb, mo, p));
    }
    profile_after(st);
    return check_launch("tc gemm");
}

template <int FORM, int BN, int CTAS, int KB = BKB, int G = EPI_GROUPS>
int launch_tc_cfg(const CUtensorMap &ma, const CUtensorMap &mb, TcParams p, int workers, cudaStream_t st)
{
    // The int32 result leaves through bulk stores where its layout allows it (16-byte aligned rows), which
    // costs the kernel one pipeline stage of shared memory; otherwise the epilogue stores from registers.
    CUtensorMap mo = ma;
    p.tma_out = 0;
    p.tiles_n = (int32_t)ceil_div(p.N, BN);
    p.idesc |= (uint32_t)(BN >> 3) << 17;
    if (CTAS == 2) p.idesc = (p.idesc & ~(0x1fu << 24)) | ((uint32_t)((2 * BM) >> 4) << 24);   // the pair's instruction is 256 rows tall
    {
        const int64_t rest = p.N - (int64_t)(p.tiles_n - 1) * BN;       // columns of the last block, 1..BN
        p.n_last = (int32_t)(rest >= BN ? BN : ((rest + 15) / 16) * 16);
        p.idesc_last = (p.idesc & ~(0x3fu << 17)) | ((uint32_t)(p.n_last >> 3) << 17);
    }
    const bool conv_full_tiles = p.conv && p.cR * p.cW == BM && p.cG == 1;
    if (p.out != nullptr && aligned(p.out, 16)) {
        // (the bulk store clips the innermost extent in 16-byte units, so N must be a whole number of them)
        if (!p.conv && p.epilogue == EPI_ROWMAJOR && p.ldo % 4 == 0 && p.N % 4 == 0) {
            cuuint64_t dims[2] = {(cuuint64_t)p.N, (cuuint64_t)p.M};
            cuuint64_t strides[1] = {(cuuint64_t)p.ldo * 4};
            cuuint32_t box[2] = {32, 32};
            if (int rc = make_map_out(&mo, CU_TENSOR_MAP_DATA_TYPE_INT32, 2, p.out, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
                return rc;
            p.tma_out = 1;
        } else if (conv_full_tiles && p.epilogue == EPI_NCHW && p.hw % 4 == 0 && p.hw == (int64_t)p.cH * p.cW) {
            cuuint64_t dims[3] = {(cuuint64_t)p.hw, (cuuint64_t)p.N, (cuuint64_t)(p.M / p.hw)};
            cuuint64_t strides[2] = {(cuuint64_t)p.hw * 4, (cuuint64_t)p.hw * 4 * (cuuint64_t)p.N};
            cuuint32_t box[3] = {32, 32, 1};
            if (int rc = make_map_out(&mo, CU_TENSOR_MAP_DATA_TYPE_INT32, 3, p.out, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE))
                return rc;
            p.tma_out = 2;
        }
    }
    if (p.tma_out) return launch_tc_stg<FORM, BN, 1, CTAS, KB, G>(ma, mb, mo, p, workers, st);
    return launch_tc_stg<FORM, BN, 0, CTAS, KB, G>(ma, mb, mo, p, workers, st);
}

// Tile width.  Measured on B200: the time of one wave of tiles depends only weakly on the width (about
// 4.2 us + 4.7 ns per column at K = 4096), because a K block costs the issuing threads and the TMA path
// about the same whatever its width.  So: fewest waves first, the width as a small correction.
int pick_bn(int64_t tiles_m, int64_t N, int workers, int min_bn)
{
    static const int cand[] = {224, 192, 128, 64, 32};
    int best = cand[0];
    double best_cost = 1e300;
    for (int i = 0; i < 5; ++i) {
        const int bn = cand[i];
        if (bn < min_bn) continue;
        const int64_t tiles = tiles_m * ceil_div(N, bn);
        const int64_t waves = ceil_div(tiles, workers);
        const double cost = (double)waves * (bn + 900);
        if (cost < best_cost - 1e-9) { best_cost = cost; best = bn; }
    }
    return best;
}

int grid_for_items(int64_t items)
{
    const int64_t need = ceil_div(items, 256);
    const int64_t cap = (int64_t)sm_count() * 32;
    return (int)(need < cap ? need : cap);
}

}  // namespace

bool tc_form_holds(int form, int planes, int mode)
{
    if (form == QNN_FORM_FP4) return planes <= 2;                       // {0..3} or {-3,-1,1,3}
    if (form == QNN_FORM_I8) return mode == QNN_MODE_PM1 ? planes <= 7 : planes <= 8;   // +-127 / 0..255
    return false;
}

int tc_pick_form(int ka, int a_mode, int kb, int b_mode, int64_t K)
{
    const int64_t la = (1 << ka) - 1, lb = (1 << kb) - 1;
    // fp32 accumulation of integer products stays exact while every partial sum is below 2^24
    if (tc_form_holds(QNN_FORM_FP4, ka, a_mode) && tc_form_holds(QNN_FORM_FP4, kb, b_mode) && K * la * lb < ((int64_t)1 << 24))
        return QNN_FORM_FP4;
    if (tc_form_holds(QNN_FORM_I8, ka, a_mode) && tc_form_holds(QNN_FORM_I8, kb, b_mode)) return QNN_FORM_I8;
    return 0;
}

int64_t tc_row_bytes(int64_t kwords, int form) { return form == QNN_FORM_FP4 ? kwords * 16 : kwords * 32; }
int64_t tc_row_pitch(int64_t kwords, int form) { return (int64_t)round_up((size_t)tc_row_bytes(kwords, form), 128); }

int tc_expand(const uint32_t *src, int planes, int mode, int64_t ld, int64_t plane_stride, int64_t rows, int64_t kwords,
              int64_t pad_period, int pad_tail, int form, uint8_t *dst, int64_t dst_ld, cudaStream_t st)
{
    if (rows == 0 || kwords == 0) return QNN_OK;
    QNN_REQUIRE(tc_form_holds(form, planes, mode), QNN_ERR_UNSUPPORTED, "tc expand: %d planes do not fit form %d", planes, form);
    const int64_t items = form == QNN_FORM_FP4 ? rows * kwords : rows * kwords * 2;
    const bool narrow = items < ((int64_t)1 << 31);
    const int grid = grid_for_items(items);
    const int pm1 = mode == QNN_MODE_PM1;
    if (form == QNN_FORM_FP4) {
        if (narrow)
            QNN_CUDA(launch_pdl(expand_fp4_kernel<uint32_t>, dim3(grid), dim3(256), 0, st, src, planes, pm1, ld, plane_stride, rows, kwords, pad_period, pad_tail, dst,
                                dst_ld));
        else
            QNN_CUDA(launch_pdl(expand_fp4_kernel<int64_t>, dim3(grid), dim3(256), 0, st, src, planes, pm1, ld, plane_stride, rows, kwords, pad_period, pad_tail, dst,
                                dst_ld));
    } else {
        if (narrow)
            QNN_CUDA(launch_pdl(expand_i8_kernel<uint32_t>, dim3(grid), dim3(256), 0, st, src, planes, pm1, ld, plane_stride, rows, kwords, pad_period, pad_tail, dst,
                                dst_ld));
        else
            QNN_CUDA(launch_pdl(expand_i8_kernel<int64_t>, dim3(grid), dim3(256), 0, st, src, planes, pm1, ld, plane_stride, rows, kwords, pad_period, pad_tail, dst,
                                dst_ld));
    }
    return check_launch("tc expand");
}

bool gemm_tc_supported(const GemmArgs &g)
{
    if (tc_pick_form(g.ka, g.a_mode, g.kb, g.b_mode, g.K) == 0) return false;
    if (g.M > (int64_t)1 << 30 || g.N > (int64_t)1 << 30) return false;
    return true;
}

size_t gemm_tc_workspace_bytes(int64_t M, int64_t N, int64_t K, int, int)
{
    const int64_t rb = tc_row_pitch(ceil_div(K, 32), QNN_FORM_I8);
    return round_up((size_t)M * (size_t)rb, 256) + round_up((size_t)N * (size_t)rb, 256);
}

int launch_gemm_tc(const GemmArgs &g, int form, void *ws, size_t ws_bytes, cudaStream_t st)
{
    const int64_t kwords = g.kwords > 0 ? g.kwords : ceil_div(g.K, 32);
    QNN_REQUIRE(kwords > 0, QNN_ERR_UNSUPPORTED, "tc gemm: K = 0 is handled by QNN_ALGO_POPC");
    const int best = tc_pick_form(g.ka, g.a_mode, g.kb, g.b_mode, g.K);
    if (form == 0) {
        form = best;
        if (g.a_tc) form = g.a_tc_form;                    // operands that already exist decide
        else if (g.b_tc) form = g.b_tc_form;
    }
    QNN_REQUIRE(form == QNN_FORM_I8 || form == QNN_FORM_FP4, QNN_ERR_UNSUPPORTED,
                "tc gemm: operand values do not fit a tensor-core form; use QNN_ALGO_POPC");
    QNN_REQUIRE(tc_form_holds(form, g.ka, g.a_mode) && tc_form_holds(form, g.kb, g.b_mode) &&
                    (form != QNN_FORM_FP4 || best == QNN_FORM_FP4),
                QNN_ERR_UNSUPPORTED, "tc gemm: operand values (%d and %d planes, K = %lld) do not fit form %d", g.ka, g.kb,
                (long long)g.K, form);
    QNN_REQUIRE((!g.a_tc || g.a_tc_form == form) && (!g.b_tc || g.b_tc_form == form), QNN_ERR_INVALID_ARG,
                "tc gemm: a prepared operand is in another form than the product uses");
    QNN_REQUIRE(g.M <= (int64_t)1 << 30 && g.N <= (int64_t)1 << 30, QNN_ERR_UNSUPPORTED, "tc gemm: M or N too large");

    const int64_t row_bytes = tc_row_bytes(kwords, form);
    QNN_REQUIRE(ceil_div(row_bytes, BKB) < ((int64_t)1 << 31), QNN_ERR_UNSUPPORTED, "tc gemm: K too large");

    // where the pad bits are: a plain matrix pads only its last word; conv rows pad the last word of every tap
    int64_t period = kwords;
    int tail = (int)(g.K - 32 * (kwords - 1));
    if (g.pad_period > 0) { period = g.pad_period; tail = g.pad_tail; }
    QNN_REQUIRE(tail >= 1 && tail <= 32, QNN_ERR_INVALID_ARG, "tc gemm: inconsistent K / kwords");

    if (g.out_form) {
        QNN_REQUIRE(g.thr != nullptr, QNN_ERR_INVALID_ARG, "tc gemm: thresholds required for a form output");
        QNN_REQUIRE(g.out_form_kind == QNN_FORM_I8 || g.out_form_kind == QNN_FORM_FP4, QNN_ERR_INVALID_ARG, "tc gemm: bad output form");
        QNN_REQUIRE(aligned(g.out_form, 16) && g.ld_form % 16 == 0 &&
                        g.ld_form >= tc_row_bytes(ceil_div(g.N, 32), g.out_form_kind),
                    QNN_ERR_ALIGNMENT, "tc gemm: form output needs a 16-byte aligned base and a row stride covering N");
    }
    if (g.conv) QNN_REQUIRE(g.a_tc != nullptr, QNN_ERR_INVALID_ARG, "tc conv: the NHWC operand must be prepared");

    // operands: use prepared ones, expand the others into the workspace (every argument check comes before this point)
    const uint8_t *a8 = static_cast<const uint8_t *>(g.a_tc);
    const uint8_t *b8 = static_cast<const uint8_t *>(g.b_tc);
    int64_t a_ld = g.a_tc_ld, b_ld = g.b_tc_ld;
    int64_t a_row_bytes = row_bytes;
    size_t need = 0;
    const int64_t pitch = tc_row_pitch(kwords, form);
    const size_t a_bytes = g.a_tc ? 0 : round_up((size_t)g.M * (size_t)pitch, 256);
    const size_t b_bytes = g.b_tc ? 0 : round_up((size_t)g.N * (size_t)pitch, 256);
    need = a_bytes + b_bytes;
    if (need > 0)
        QNN_REQUIRE(ws != nullptr && aligned(ws, 256) && ws_bytes >= need, QNN_ERR_WORKSPACE,
                    "tc gemm: workspace of at least %zu bytes (256-byte aligned) required", need);
    if (g.a_tc) {
        QNN_REQUIRE(aligned(g.a_tc, 16) && a_ld % 16 == 0 && a_ld > 0, QNN_ERR_ALIGNMENT,
                    "tc gemm: prepared A operand needs a 16-byte aligned base and row stride");
        if (!g.conv && a_ld < row_bytes) a_row_bytes = a_ld;           // e.g. raw uint8 codes: K bytes per row, rest reads 0
    } else {
        QNN_REQUIRE(!g.conv, QNN_ERR_INVALID_ARG, "tc conv: the NHWC operand must be prepared");
        uint8_t *dst = static_cast<uint8_t *>(ws);
        if (int rc = tc_expand(g.a, g.ka, g.a_mode, g.lda, g.a_plane_stride, g.M, kwords, period, tail, form, dst, pitch, st))
            return rc;
        a8 = dst; a_ld = pitch;
    }
    if (g.b_tc) {
        QNN_REQUIRE(aligned(g.b_tc, 16) && b_ld % 16 == 0 && b_ld >= row_bytes, QNN_ERR_ALIGNMENT,
                    "tc gemm: prepared B operand needs a 16-byte aligned base and row stride");
    } else {
        uint8_t *dst = static_cast<uint8_t *>(ws) + a_bytes;
        if (int rc = tc_expand(g.b, g.kb, g.b_mode, g.ldb, g.b_plane_stride, g.N, kwords, period, tail, form, dst, pitch, st))
            return rc;
        b8 = dst; b_ld = pitch;
    }

    TcParams p{};
    p.M = g.M; p.N = g.N; p.num_kb = (int32_t)ceil_div(row_bytes, BKB);
    p.tiles_m = (int32_t)ceil_div(g.M, BM);
    p.a_tx_bytes = BM * BKB;
    p.epilogue = g.epilogue; p.out = g.out; p.ldo = g.ldo; p.hw = g.hw > 0 ? g.hw : 1;
    p.thr = g.thr; p.flip = g.flip; p.out_bits = g.out_bits; p.ld_bits = g.ld_bits;
    p.out_form = static_cast<uint8_t *>(g.out_form); p.ld_form = g.ld_form; p.out_form_kind = g.out_form_kind;
    {
        const int64_t maxsum = g.K * ((1 << g.ka) - 1) * (int64_t)((1 << g.kb) - 1);
        p.thr_clamp = maxsum + 1 < ((int64_t)1 << 30) ? (int32_t)(maxsum + 1) : 0;
    }
    if (form == QNN_FORM_FP4) {
        // block-scaled instruction descriptor: A and B e2m1 (format 1), both K-major, ue8m0 scales, M = 128
        p.idesc = (1u << 7) | (1u << 10) | (1u << 23) | ((uint32_t)(BM >> 4) << 24);
    } else {
        // int32 accumulator, A/B int8 signed (PM1) or unsigned (U01), both K-major, M = 128
        p.idesc = (2u << 4) | ((g.a_mode == QNN_MODE_PM1 ? 1u : 0u) << 7) | ((g.b_mode == QNN_MODE_PM1 ? 1u : 0u) << 10) |
                  ((uint32_t)(BM >> 4) << 24);
    }

    CUtensorMap ma, mb;
    // channel blocks of 64 bytes (128 e2m1 channels): the convolution's K block shrinks with them
    const int kblk = (g.conv && g.conv->kblk == 64) ? 64 : BKB;
    QNN_REQUIRE(kblk == BKB || form == QNN_FORM_FP4, QNN_ERR_INVALID_ARG, "tc conv: 64-byte channel blocks are an e2m1 layout");
    if (g.conv) {
        const ConvImplicit &c = *g.conv;
        QNN_REQUIRE(c.W >= 1 && c.W <= BM && c.KH == 2 * c.pad + 1 && c.KW == 2 * c.pad + 1 && c.pad <= 3,
                    QNN_ERR_UNSUPPORTED, "tc conv: implicit path needs a stride-1 'same' filter and W <= 128");
        const int R = BM / c.W < c.H ? BM / c.W : c.H;                  // image rows per tile
        QNN_REQUIRE(R >= 1 && R <= 256, QNN_ERR_UNSUPPORTED, "tc conv: bad tile height");
        // feature maps of at most half a tile: several whole images per tile
        const int G = (R == c.H && BM / (c.H * c.W) >= 2) ? BM / (c.H * c.W) : 1;
        p.conv = 1; p.cH = c.H; p.cW = c.W; p.cR = R; p.tiles_per_img = (int32_t)ceil_div(c.H, R);
        p.cG = G; p.cB = c.B;
        if (c.pool) {
            QNN_REQUIRE((c.W == 2 || c.W == 4 || c.W == 8 || c.W == 16) && c.H % 2 == 0 && (R % 2 == 0) && g.out == nullptr,
                        QNN_ERR_UNSUPPORTED, "tc conv: pooling inside the epilogue needs W in {2,4,8,16}, an even H and no int32 output");
            p.pool = 1;
        }
        p.cKW = c.KW; p.cpad = c.pad; p.cblocks = c.cblocks; p.corr = c.corr; p.corr_ld = (int64_t)round_up((size_t)g.N, 32);
        QNN_REQUIRE(aligned(c.corr, 16), QNN_ERR_ALIGNMENT, "tc conv: correction table must be 16-byte aligned");
        p.tiles_m = (int32_t)ceil_div(c.B, G) * p.tiles_per_img;
        p.a_tx_bytes = G * R * c.W * kblk;
        p.num_kb = (int32_t)ceil_div(row_bytes, kblk);
        QNN_REQUIRE(p.num_kb == c.KH * c.KW * c.cblocks, QNN_ERR_INVALID_ARG, "tc conv: K blocks do not match the filter");
        QNN_REQUIRE(g.M == (int64_t)c.B * c.H * c.W, QNN_ERR_INVALID_ARG, "tc conv: M does not match the image geometry");
        QNN_REQUIRE(a_ld == (int64_t)c.cblocks * kblk, QNN_ERR_INVALID_ARG, "tc conv: pixels must be whole channel blocks apart");
        if (int rc = make_map_nhwc(&ma, a8, c.B, c.H, c.W, (int64_t)c.cblocks * kblk, R, G, kblk)) return rc;
    } else {
        if (int rc = make_map_2d(&ma, a8, g.M, a_row_bytes, a_ld, BM)) return rc;
    }
    // Large plain products with a long K run on CTA pairs (cta_group::2): one 256 x BN tile per pair halves, per
    // SM, both the operand bytes to load and the instructions to issue.  Measured on B200: 8192^3 with int32
    // output 209 -> 182 us, 10000 x 4096 x 4096 68 -> 66 us; with fewer than a dozen K blocks per tile the
    // cross-SM hand-offs cost more than the pair saves (10000 x 4096 x 784: 41 -> 47 us), so those stay on single
    // CTAs.  QNN_TC_PAIRS=0 in the environment keeps single CTAs everywhere.
    static const bool pairs_off = [] { const char *e = getenv("QNN_TC_PAIRS"); return e && e[0] == '0'; }();
    const int pairs_resident = pairs_off ? 0 : pairs_resident_on_current_device();
    const int64_t tiles_m2 = ceil_div(g.M, 2 * BM);
    static const int pair_min_kb = [] { const char *e = getenv("QNN_TC_PAIR_MIN_KB"); return e ? atoi(e) : 12; }();
    const bool pairs = !g.conv && pairs_resident >= 8 && p.num_kb >= pair_min_kb && tiles_m2 * ceil_div(g.N, 224) >= pairs_resident;
    if (pairs) {
        p.tiles_m = (int32_t)tiles_m2;
        int bn = pick_bn(tiles_m2, g.N, pairs_resident, 64);
        if (form == QNN_FORM_I8 && bn == 224) {
            // (int8 has no scale columns in tensor memory: two 256-column accumulator stages fit)
            const int64_t w224 = ceil_div(tiles_m2 * ceil_div(g.N, 224), pairs_resident), w256 = ceil_div(tiles_m2 * ceil_div(g.N, 256), pairs_resident);
            if (w256 * (256 + 900) < w224 * (224 + 900)) bn = 256;
        }
        if (int rc = make_map_2d(&mb, b8, g.N, row_bytes, b_ld, bn / 2)) return rc;
        if (form == QNN_FORM_FP4) {
            switch (bn) {
                case 224: return launch_tc_cfg<QNN_FORM_FP4, 224, 2>(ma, mb, p, pairs_resident, st);
                case 192: return launch_tc_cfg<QNN_FORM_FP4, 192, 2>(ma, mb, p, pairs_resident, st);
                case 128: return launch_tc_cfg<QNN_FORM_FP4, 128, 2>(ma, mb, p, pairs_resident, st);
                default: return launch_tc_cfg<QNN_FORM_FP4, 64, 2>(ma, mb, p, pairs_resident, st);
            }
        }
        switch (bn) {
            case 256: return launch_tc_cfg<QNN_FORM_I8, 256, 2>(ma, mb, p, pairs_resident, st);
            case 224: return launch_tc_cfg<QNN_FORM_I8, 224, 2>(ma, mb, p, pairs_resident, st);
            case 192: return launch_tc_cfg<QNN_FORM_I8, 192, 2>(ma, mb, p, pairs_resident, st);
            case 128: return launch_tc_cfg<QNN_FORM_I8, 128, 2>(ma, mb, p, pairs_resident, st);
            default: return launch_tc_cfg<QNN_FORM_I8, 64, 2>(ma, mb, p, pairs_resident, st);
        }
    }

    // Short K on the int8 form (Algorithm 4's first layer, K = 784): single CTAs are bound there by the bytes an SM takes
    // from L2 (48 KB per K block at 256 columns) and the pair halves the B share of them, but with 4 .. 11 K blocks per
    // tile the pair's epilogue sets the pace -- so the pair runs with three epilogue warps per accumulator quarter
    // (measured on 10000 x 4096 x 784: single CTAs 37.4-39.3 us, pairs 37.1 us, pairs with three warps 35.3 us).
    // QNN_TC_PAIRS_SHORT=0 in the environment keeps single CTAs.
    static const bool pairs_short_off = [] { const char *e = getenv("QNN_TC_PAIRS_SHORT"); return e && e[0] == '0'; }();
    if (!pairs_short_off && !g.conv && form == QNN_FORM_I8 && pairs_resident >= 8 && p.num_kb >= 4 && p.num_kb < pair_min_kb &&
        g.N >= 256 && tiles_m2 * ceil_div(g.N, 256) >= 2 * (int64_t)pairs_resident) {
        p.tiles_m = (int32_t)tiles_m2;
        if (int rc = make_map_2d(&mb, b8, g.N, row_bytes, b_ld, 128)) return rc;
        return launch_tc_cfg<QNN_FORM_I8, 256, 2, BKB, 3>(ma, mb, p, pairs_resident, st);
    }

    // (int8 has no scale columns in tensor memory, so two 256-column accumulator stages fit: tried for wide single-CTA products)
    int bn = pick_bn(p.tiles_m, g.N, sm_count(), 32);
    if (form == QNN_FORM_I8 && !g.conv && kblk == BKB && bn == 224) {
        const int64_t w224 = ceil_div(p.tiles_m * ceil_div(g.N, 224), sm_count()), w256 = ceil_div(p.tiles_m * ceil_div(g.N, 256), sm_count());
        if (w256 * (256 + 900) < w224 * (224 + 900)) bn = 256;
    }
    if (int rc = make_map_2d(&mb, b8, g.N, row_bytes, b_ld, bn, kblk)) return rc;
    if (kblk == 64) {
        switch (bn) {
            case 224: return launch_tc_cfg<QNN_FORM_FP4, 224, 1, 64>(ma, mb, p, sm_count(), st);
            case 192: return launch_tc_cfg<QNN_FORM_FP4, 192, 1, 64>(ma, mb, p, sm_count(), st);
            case 128: return launch_tc_cfg<QNN_FORM_FP4, 128, 1, 64>(ma, mb, p, sm_count(), st);
            case 64: return launch_tc_cfg<QNN_FORM_FP4, 64, 1, 64>(ma, mb, p, sm_count(), st);
            default: return launch_tc_cfg<QNN_FORM_FP4, 32, 1, 64>(ma, mb, p, sm_count(), st);
        }
    }
    if (form == QNN_FORM_FP4) {
        switch (bn) {
            case 224: return launch_tc_cfg<QNN_FORM_FP4, 224, 1>(ma, mb, p, sm_count(), st);
            case 192: return launch_tc_cfg<QNN_FORM_FP4, 192, 1>(ma, mb, p, sm_count(), st);
            case 128: return launch_tc_cfg<QNN_FORM_FP4, 128, 1>(ma, mb, p, sm_count(), st);
            case 64: return launch_tc_cfg<QNN_FORM_FP4, 64, 1>(ma, mb, p, sm_count(), st);
            default: return launch_tc_cfg<QNN_FORM_FP4, 32, 1>(ma, mb, p, sm_count(), st);
        }
    }
    switch (bn) {
        case 256: return launch_tc_cfg<QNN_FORM_I8, 256, 1>(ma, mb, p, sm_count(), st);
        case 224: return launch_tc_cfg<QNN_FORM_I8, 224, 1>(ma, mb, p, sm_count(), st);
        case 192: return launch_tc_cfg<QNN_FORM_I8, 192, 1>(ma, mb, p, sm_count(), st);
        case 128: return launch_tc_cfg<QNN_FORM_I8, 128, 1>(ma, mb, p, sm_count(), st);
        case 64: return launch_tc_cfg<QNN_FORM_I8, 64, 1>(ma, mb, p, sm_count(), st);
        default: return launch_tc_cfg<QNN_FORM_I8, 32, 1>(ma, mb, p, sm_count(), st);
    }
}

}  // namespace qnn

// ---- issue-only pipe measurements ------------------------------------------------------------------------------
//
// What the pipes can do when nothing else is in the way: every CTA multiplies ONE resident shared-memory tile pair
// over and over (no loads, no epilogue), or runs xor / popc / add on registers.  The bench divides the operations by
// the device time of such a launch and reports the product kernels against that figure as well.
namespace qnn {
namespace {

constexpr int PEAK_N = 256;             // instruction shape of the tensor measurement: 128 x 256 x (32 bytes of K)

template <int FORM>
__global__ void __launch_bounds__(128, 1) tc_peak_kernel(int iters, uint32_t idesc, int *ok_out)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - raw);
    constexpr int A_BYTES = BM * BKB, B_BYTES = PEAK_N * BKB;
    uint64_t *bar = reinterpret_cast<uint64_t *>(gen + A_BYTES + B_BYTES);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5;
    // operand values: A all +1, B +1 / -1 alternating along K, so that every K step adds zero to the accumulators
    const uint32_t a_word = FORM == QNN_FORM_FP4 ? 0x22222222u : 0x01010101u;
    const uint32_t b_word = FORM == QNN_FORM_FP4 ? 0xA2A2A2A2u : 0xFF01FF01u;
    for (int i = threadIdx.x; i < A_BYTES / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(gen)[i] = a_word;
    for (int i = threadIdx.x; i < B_BYTES / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(gen + A_BYTES)[i] = b_word;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(bar), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    fence_async_shared();
    if (warp == 0) tmem_alloc<1>(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (FORM == QNN_FORM_FP4) {
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_st8(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(PEAK_N + 8 * c), 0x7f7f7f7fu);
        tmem_st_wait();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    if (threadIdx.x == 0) {
        const uint64_t da = make_kmajor_desc<BKB>(base), db = make_kmajor_desc<BKB>(base + A_BYTES);
        const uint32_t sf = tmem_base + (uint32_t)PEAK_N;
        for (int it = 0; it < iters; ++it) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const uint64_t a = da + (uint64_t)(2 * ks), b = db + (uint64_t)(2 * ks);
                const uint32_t acc = (it | ks) != 0;
                if (FORM == QNN_FORM_FP4)
                    asm volatile("{\n.reg .pred P;\nsetp.ne.b32 P, %4, 0;\n"
                                 "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%5], P;\n}\n"
                                 ::"r"(tmem_base), "l"(a), "l"(b), "r"(idesc), "r"(acc), "r"(sf) : "memory");
                else
                    asm volatile("{\n.reg .pred P;\nsetp.ne.b32 P, %4, 0;\n"
                                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, P;\n}\n"
                                 ::"r"(tmem_base), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
            }
        }
        umma_commit(smem_u32(bar));
        const bool done = mbar_wait(smem_u32(bar), 0, abort_flag, 8);
        if (blockIdx.x == 0 && ok_out != nullptr) *ok_out = done ? 1 : 0;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) tmem_dealloc<1>(tmem_base, 512);
}

// xor, popc, add on registers: eight independent chains per thread (Eq. 11's three instructions, nothing else)
__global__ void __launch_bounds__(1024) popc_peak_kernel(int iters, uint32_t seed, uint32_t *sink)
{
    uint32_t x[8], acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { x[i] = seed * (threadIdx.x + 1) + i * 0x9e3779b9u; acc[i] = 0; }
    uint32_t y = seed ^ blockIdx.x;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] += __popc(x[i] ^ y);
        y = y * 1664525u + 1013904223u;
    }
    uint32_t t = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) t += acc[i];
    if (t == 0xffffffffu) *sink = t;         // (never true for these counts; keeps the loop alive)
}

}  // namespace
}  // namespace qnn

extern "C" int qnn_pipe_peak_launch(int pipe, int iters, double *ops_host, void *stream)
{
    using namespace qnn;
    QNN_REQUIRE(iters >= 1 && iters <= (1 << 20), QNN_ERR_INVALID_ARG, "qnn_pipe_peak_launch: iters must be in 1..2^20");
    QNN_REQUIRE(ops_host != nullptr, QNN_ERR_INVALID_ARG, "qnn_pipe_peak_launch: ops_host is NULL");
    cudaStream_t st = as_stream(stream);
    const int sms = sm_count();
    if (pipe == QNN_PIPE_POPC) {
        const int blocks = 2 * sms;
        popc_peak_kernel<<<blocks, 1024, 0, st>>>(iters, 0x12345u, nullptr);
        *ops_host = 64.0 * 8.0 * (double)iters * 1024.0 * blocks;          // one 32-bit xor/popc/add = 32 products = 64 operations
        return check_launch("qnn_pipe_peak_launch");
    }
    QNN_REQUIRE(pipe == QNN_PIPE_TENSOR_FP4 || pipe == QNN_PIPE_TENSOR_I8, QNN_ERR_INVALID_ARG, "qnn_pipe_peak_launch: unknown pipe %d", pipe);
    const size_t smem = (size_t)BM * BKB + (size_t)PEAK_N * BKB + 64 + 1024;
    const int kstep = pipe == QNN_PIPE_TENSOR_FP4 ? 64 : 32;               // elements of K per instruction (32 bytes)
    *ops_host = 2.0 * BM * PEAK_N * kstep * 4.0 * (double)iters * sms;
    if (pipe == QNN_PIPE_TENSOR_FP4) {
        const uint32_t idesc = (1u << 7) | (1u << 10) | (1u << 23) | ((uint32_t)(BM >> 4) << 24) | ((uint32_t)(PEAK_N >> 3) << 17);
        QNN_CUDA(cudaFuncSetAttribute(tc_peak_kernel<QNN_FORM_FP4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        tc_peak_kernel<QNN_FORM_FP4><<<sms, 128, smem, st>>>(iters, idesc, nullptr);
    } else {
        const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BM >> 4) << 24) | ((uint32_t)(PEAK_N >> 3) << 17);
        QNN_CUDA(cudaFuncSetAttribute(tc_peak_kernel<QNN_FORM_I8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        tc_peak_kernel<QNN_FORM_I8><<<sms, 128, smem, st>>>(iters, idesc, nullptr);
    }
    return check_launch("qnn_pipe_peak_launch");
}

extern "C" int qnn_selftest_wait_timeout(void *stream)
{
    using namespace qnn;
    wait_probe_kernel<<<1, 32, 0, as_stream(stream)>>>();
    return check_launch("qnn_selftest_wait_timeout");
}

extern "C" int qnn_device_status(void *stream)
{
    using namespace qnn;
    QNN_CUDA(cudaStreamSynchronize(as_stream(stream)));
    int code = 0, code_fc = 0, code_sm = 0;
    QNN_CUDA(status_read_clear(&code));
    if (int rc = fc_f32_status(&code_fc)) return rc;
    if (int rc = smallm_status(&code_sm)) return rc;
    if (code == 0) code = code_fc;
    if (code == 0) code = code_sm;
    if (code != 0) return fail(QNN_ERR_TIMEOUT, "a bounded device-side wait ran out (wait site %d)", code);
    return QNN_OK;
}
