// Tensor-core matrix products (placeholder until the tcgen05 path lands).
#include "qnn_internal.cuh"

namespace qnn {

bool gemm_tc_supported(const GemmArgs &) { return false; }
size_t gemm_tc_workspace_bytes(int64_t, int64_t, int64_t, int, int) { return 0; }
int launch_gemm_tc(const GemmArgs &, void *, size_t, cudaStream_t)
{
    return fail(QNN_ERR_UNSUPPORTED, "tcgen05 int8 path is not built yet");
}
int launch_gemm_b1mma(const GemmArgs &, cudaStream_t)
{
    return fail(QNN_ERR_UNSUPPORTED, "1-bit mma.sync path is not built yet");
}

}  // namespace qnn

extern "C" int qnn_device_status(void *stream)
{
    cudaError_t e = cudaStreamSynchronize(qnn::as_stream(stream));
    if (e != cudaSuccess) return qnn::fail(QNN_ERR_CUDA, "qnn_device_status: %s", cudaGetErrorString(e));
    return QNN_OK;
}
