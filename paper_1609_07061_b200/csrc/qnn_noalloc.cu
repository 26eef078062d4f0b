// qnn_xnor_gemm_noalloc: the tensor-core XNOR product for callers that cannot obtain
// device memory at call time.  Its int8 operand scratch is a fixed array that is
// part of the loaded library image instead of a caller workspace.
#include <mutex>
#include "qnn_internal.cuh"

namespace qnn {
namespace {

// Lives in every CUDA context that loads this library, from load until the process
// exits.  Shared by all calls; holds whatever the last call left in it.
static __device__ __align__(256) uint8_t g_noalloc_scratch[QNN_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices] = {};     // device address of g_noalloc_scratch, per device ordinal

// In host code the array's name is only a handle for the runtime, not an address a
// kernel may use: the per-device address has to be asked for, with that device current.
// The address is kept per device ordinal for the life of the process; it does not
// survive cudaDeviceReset (a process that resets a device must not call this entry
// point on it again).
int scratch_for_current_device(void **out)
{
    int dev = 0;
    QNN_CUDA(cudaGetDevice(&dev));
    QNN_REQUIRE(dev >= 0 && dev < kMaxDevices, QNN_ERR_UNSUPPORTED, "qnn_xnor_gemm_noalloc: device ordinal %d not supported", dev);
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || p == nullptr)
            return fail(QNN_ERR_CUDA, "qnn_xnor_gemm_noalloc: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return QNN_OK;
}

}  // namespace
}  // namespace qnn

using namespace qnn;

extern "C" int qnn_xnor_gemm_noalloc(const uint32_t *a, int64_t lda, const uint32_t *b, int64_t ldb, int64_t M, int64_t N,
                                     int64_t K, int32_t *out, int64_t ldo, void *stream)
{
    GemmArgs g{};
    g.a = a; g.b = b; g.lda = lda; g.ldb = ldb; g.ka = g.kb = 1; g.a_mode = g.b_mode = QNN_MODE_PM1;
    g.M = M; g.N = N; g.K = K; g.epilogue = EPI_ROWMAJOR; g.out = out; g.ldo = ldo;
    QNN_REQUIRE(out != nullptr || M == 0 || N == 0, QNN_ERR_INVALID_ARG, "qnn_xnor_gemm_noalloc: out is NULL");
    if (int rc = validate_gemm(g)) return rc;
    if (M == 0 || N == 0) return QNN_OK;
    // An empty sum: every output is 0, as qnn_xnor_gemm gives.  The CUDA-core kernel writes it and needs no scratch.
    if (K == 0) return run_gemm(g, QNN_ALGO_POPC, nullptr, 0, as_stream(stream));
    const size_t need = gemm_tc_workspace_bytes(M, N, K, 1, 1);
    QNN_REQUIRE(need <= (size_t)QNN_NOALLOC_SCRATCH_BYTES, QNN_ERR_WORKSPACE,
                "qnn_xnor_gemm_noalloc: this shape needs %zu bytes of operand scratch but the built-in array holds %zu; "
                "use qnn_xnor_gemm with a caller workspace", need, (size_t)QNN_NOALLOC_SCRATCH_BYTES);
    void *scratch = nullptr;
    if (int rc = scratch_for_current_device(&scratch)) return rc;
    // Every byte the product kernel reads from the scratch is rewritten by this call's expansion
    // passes first (pad positions included), so nothing has to be cleared between calls.
    return launch_gemm_tc(g, QNN_FORM_I8, scratch, (size_t)QNN_NOALLOC_SCRATCH_BYTES, as_stream(stream));
}
