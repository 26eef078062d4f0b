// Internal helpers shared by the library's translation units (host-side error
// plumbing, small device utilities).  Not part of the ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "qnn.h"

namespace qnn {

// Records a formatted message in the thread-local error slot and returns `code`.
int fail(int code, const char *fmt, ...);
void clear_error();
// Leaves a text in the same slot without failing the call (e.g. when QNN_ALGO_AUTO had to take a slower algorithm).
void note(const char *fmt, ...);

inline cudaStream_t as_stream(void *s) { return reinterpret_cast<cudaStream_t>(s); }
inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t round_up(size_t a, size_t b) { return (a + b - 1) / b * b; }

// Launch check: converts a pending launch error into QNN_ERR_CUDA.
int check_launch(const char *what);

#define QNN_REQUIRE(cond, code, ...)                     \
    do {                                                 \
        if (!(cond)) return ::qnn::fail((code), __VA_ARGS__); \
    } while (0)

#define QNN_CUDA(call)                                                                   \
    do {                                                                                 \
        cudaError_t e__ = (call);                                                        \
        if (e__ != cudaSuccess)                                                          \
            return ::qnn::fail(QNN_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e__)); \
    } while (0)

int sm_count();

// Armed measurement events (see qnn_set_kernel_events): call around the product kernel launch.
void profile_before(cudaStream_t st);
void profile_after(cudaStream_t st);

// ---- internal launchers shared between translation units -------------------

enum Epilogue { EPI_ROWMAJOR = 0, EPI_NCHW = 1, EPI_BITS = 2 };

// Implicit-GEMM view of a stride-1 "same" convolution for the tensor-core path: the A operand is the
// NHWC activation tensor in tensor-core form, read tap by tap through a 4-D tensor map whose
// out-of-image reads return zero; `corr` adds back what the padding value contributes.
struct ConvImplicit {
    int32_t B, H, W, KH, KW, pad;
    int32_t cblocks;            // channel blocks per pixel
    int32_t kblk;               // bytes per channel block: 128 (0 means 128), or 64 for 128 e2m1 channels
    int32_t pool;               // 1: the epilogue max-pools the thresholded signs 2 x 2 (outputs are [B, H/2, W/2, ...])
    const int32_t *corr;        // [(pad+1)^4][N rounded up to 32] border corrections (pad columns and class 0 zero)
};

struct GemmArgs {
    const uint32_t *a;      // ka planes [M, lda]
    const uint32_t *b;      // kb planes [N, ldb]
    int64_t lda, ldb, a_plane_stride, b_plane_stride;
    int ka, kb, a_mode, b_mode;
    int64_t M, N, K;        // K = number of real products per output (sets the constant term)
    int64_t kwords;         // words per row to reduce over; 0 = ceil(K/32) (conv rows carry interior pad bits)
    int64_t pad_period;     // > 0: every pad_period-th word holds only pad_tail valid bits (conv: words per tap)
    int pad_tail;
    int epilogue;           // Epilogue
    int32_t *out;           // EPI_ROWMAJOR / EPI_NCHW
    int64_t ldo;            // EPI_ROWMAJOR
    int64_t hw;             // EPI_NCHW: spatial size Ho*Wo (row m = b*hw + p -> out[b, n, p])
    const int32_t *thr;     // EPI_BITS (or EPI_NCHW + bits when out_bits != nullptr)
    const uint8_t *flip;
    uint32_t *out_bits;     // EPI_BITS: [M, ld_bits]
    int64_t ld_bits;
    // ---- tensor-core extras (all optional) ----
    const void *a_tc;       // A already in tensor-core form (QNN_FORM_*), rows a_tc_ld bytes apart
    int a_tc_form;
    int64_t a_tc_ld;
    const void *b_tc;       // B likewise
    int b_tc_form;
    int64_t b_tc_ld;
    void *out_form;         // thresholded signs written as the next product's A operand in form out_form_kind
    int out_form_kind;
    int64_t ld_form;        // bytes between rows of out_form
    const ConvImplicit *conv;   // non-null: A is an NHWC tensor read as an implicit im2col
};

int validate_gemm(const GemmArgs &g);
int launch_gemm_popc(const GemmArgs &g, cudaStream_t st);
int launch_gemm_b1mma(const GemmArgs &g, cudaStream_t st);
// form: QNN_FORM_I8, QNN_FORM_FP4, or 0 = the best form the operands allow
int launch_gemm_tc(const GemmArgs &g, int form, void *ws, size_t ws_bytes, cudaStream_t st);
// upper bound over the forms (the int8 form is the larger one)
size_t gemm_tc_workspace_bytes(int64_t M, int64_t N, int64_t K, int ka, int kb);
bool gemm_tc_supported(const GemmArgs &g);
// best tensor-core form for the operand value sets (0 = none)
int tc_pick_form(int ka, int a_mode, int kb, int b_mode, int64_t K);
bool tc_form_holds(int form, int planes, int mode);
int64_t tc_row_bytes(int64_t kwords, int form);
// distance between rows the library itself lays operands out with: whole 128-byte lines, so that every TMA box row
// is one line (a row pitch that is not a multiple of 128 doubles the memory requests of the loads)
int64_t tc_row_pitch(int64_t kwords, int form);
// Prepared filter bank of the implicit tensor-core convolution: weights in tensor-core form, then the border table.
struct ConvPrep {
    int form;
    int kblk;                   // bytes of one channel block of a pixel (128, or 64: 128 e2m1 channels)
    int64_t kwords, w_pitch;
    int classes, corr_ld;
    size_t w_bytes, c_bytes;
};
bool conv_prep_layout(int Cout, int C, int KH, int KW, int pad, int want_form, ConvPrep *l);
int tc_expand(const uint32_t *src, int planes, int mode, int64_t ld, int64_t plane_stride, int64_t rows, int64_t kwords,
              int64_t pad_period, int pad_tail, int form, uint8_t *dst, int64_t dst_ld, cudaStream_t st);
int run_gemm(const GemmArgs &g, int algo, void *ws, size_t ws_bytes, cudaStream_t st);
// Small-batch product straight from packed planes (packed tiles by TMA, expanded in shared memory): no workspace.
bool gemm_smallm_supported(const GemmArgs &g);
int launch_gemm_smallm(const GemmArgs &g, cudaStream_t st);
int smallm_status(int *code);
// status word of the real-valued-weights layer kernel's bounded waits (its own translation unit): reads and clears it
int fc_f32_status(int *code);

#ifdef __CUDACC__
// Programmatic dependent launch.  A kernel launched through launch_pdl may be scheduled while the kernel before it in the
// stream is still draining; it must not touch that kernel's results (or buffers that kernel still reads) before
// griddep_wait() returns, which is when every earlier kernel has completed and its writes are visible.
// griddep_launch_dependents() lets the kernel after this one be scheduled early in the same way.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// QNN_PDL=0 in the environment launches everything with plain stream ordering.
bool pdl_enabled();

template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// bit i of the low byte of x -> bit 4*i (one bit per nibble)
__device__ __forceinline__ uint32_t spread_bits_to_nibbles(uint32_t x)
{
    x = (x | (x << 12)) & 0x000F000Fu;
    x = (x | (x << 6)) & 0x03030303u;
    x = (x | (x << 3)) & 0x11111111u;
    return x;
}
// bit i of the low nibble of x -> bit 8*i (one bit per byte)
__device__ __forceinline__ uint32_t spread_bits_to_bytes(uint32_t nib) { return (nib * 0x00204081u) & 0x01010101u; }

// 32 sign bits as 32 e2m1 values (+1 -> 0x2, -1 -> 0xA; elements outside `valid` -> 0), element 2i in the low nibble of byte i
__device__ __forceinline__ uint4 signs_to_fp4(uint32_t w, uint32_t valid)
{
    uint32_t o[4];
#pragma unroll
    for (int b = 0; b < 4; ++b)
        o[b] = (0xAAAAAAAAu ^ (spread_bits_to_nibbles((w >> (8 * b)) & 0xffu) << 3)) &
               (spread_bits_to_nibbles((valid >> (8 * b)) & 0xffu) * 0xfu);
    return make_uint4(o[0], o[1], o[2], o[3]);
}
// 32 sign bits as 32 int8 values (+1 -> 0x01, -1 -> 0xFF; elements outside `valid` -> 0): bytes 0..15 and 16..31
__device__ __forceinline__ void signs_to_i8(uint32_t w, uint32_t valid, uint4 &lo, uint4 &hi)
{
    uint32_t o[8];
#pragma unroll
    for (int b = 0; b < 8; ++b)
        o[b] = (0xFFFFFFFFu ^ (spread_bits_to_bytes((w >> (4 * b)) & 0xfu) * 0xfeu)) &
               (spread_bits_to_bytes((valid >> (4 * b)) & 0xfu) * 0xffu);
    lo = make_uint4(o[0], o[1], o[2], o[3]);
    hi = make_uint4(o[4], o[5], o[6], o[7]);
}
#endif

}  // namespace qnn
