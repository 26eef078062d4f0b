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
};

int validate_gemm(const GemmArgs &g);
int launch_gemm_popc(const GemmArgs &g, cudaStream_t st);
int launch_gemm_b1mma(const GemmArgs &g, cudaStream_t st);
int launch_gemm_tc(const GemmArgs &g, void *ws, size_t ws_bytes, cudaStream_t st);
size_t gemm_tc_workspace_bytes(int64_t M, int64_t N, int64_t K, int ka, int kb);
bool gemm_tc_supported(const GemmArgs &g);
int run_gemm(const GemmArgs &g, int algo, void *ws, size_t ws_bytes, cudaStream_t st);

}  // namespace qnn
