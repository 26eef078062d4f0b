// Host front of the matrix products: validation, algorithm selection and the
// extern "C" entry points (xnor / bit-plane, int32 or thresholded-bits output).
#include <cstdlib>
#include <cstring>
#include "qnn_internal.cuh"

namespace qnn {

int validate_gemm(const GemmArgs &g)
{
    QNN_REQUIRE(g.M >= 0 && g.N >= 0 && g.K >= 0, QNN_ERR_INVALID_ARG, "gemm: negative size");
    QNN_REQUIRE(g.K < (int64_t)1 << 31, QNN_ERR_INVALID_ARG, "gemm: K must be below 2^31");
    QNN_REQUIRE(g.ka >= 1 && g.ka <= 8 && g.kb >= 1 && g.kb <= 8, QNN_ERR_INVALID_ARG, "gemm: plane counts must be in 1..8");
    QNN_REQUIRE((g.a_mode == QNN_MODE_U01 || g.a_mode == QNN_MODE_PM1) &&
                    (g.b_mode == QNN_MODE_U01 || g.b_mode == QNN_MODE_PM1),
                QNN_ERR_INVALID_ARG, "gemm: unknown operand mode");
    const int64_t la = (1 << g.ka) - 1, lb = (1 << g.kb) - 1;
    QNN_REQUIRE(g.K == 0 || la * lb <= (((int64_t)1 << 31) - 1) / g.K, QNN_ERR_OVERFLOW,
                "gemm: K * (2^ka - 1) * (2^kb - 1) = %lld * %lld * %lld does not fit int32", (long long)g.K,
                (long long)la, (long long)lb);
    if (g.M == 0 || g.N == 0) return QNN_OK;
    const int64_t kw = g.kwords > 0 ? g.kwords : ceil_div(g.K, 32);
    QNN_REQUIRE(g.out != nullptr || g.out_bits != nullptr, QNN_ERR_INVALID_ARG, "gemm: no output buffer");
    if (g.K > 0) {
        QNN_REQUIRE(g.a && g.b, QNN_ERR_INVALID_ARG, "gemm: NULL operand");
        QNN_REQUIRE(g.lda >= kw && g.ldb >= kw, QNN_ERR_INVALID_ARG, "gemm: lda/ldb smaller than ceil(K/32)");
        QNN_REQUIRE(g.ka == 1 || g.a_plane_stride >= g.M * g.lda, QNN_ERR_INVALID_ARG, "gemm: a_plane_stride too small");
        QNN_REQUIRE(g.kb == 1 || g.b_plane_stride >= g.N * g.ldb, QNN_ERR_INVALID_ARG, "gemm: b_plane_stride too small");
        QNN_REQUIRE(aligned(g.a, 4) && aligned(g.b, 4), QNN_ERR_ALIGNMENT, "gemm: operands must be 4-byte aligned");
    }
    if (g.out) {
        QNN_REQUIRE(aligned(g.out, 4), QNN_ERR_ALIGNMENT, "gemm: out must be 4-byte aligned");
        if (g.epilogue == EPI_ROWMAJOR) QNN_REQUIRE(g.ldo >= g.N, QNN_ERR_INVALID_ARG, "gemm: ldo smaller than N");
        if (g.epilogue == EPI_NCHW) QNN_REQUIRE(g.hw >= 1 && g.M % g.hw == 0, QNN_ERR_INVALID_ARG, "gemm: bad spatial size");
    }
    if (g.out_bits) {
        QNN_REQUIRE(g.thr != nullptr, QNN_ERR_INVALID_ARG, "gemm: thresholds required for packed-bit output");
        QNN_REQUIRE(g.ld_bits >= ceil_div(g.N, 32), QNN_ERR_INVALID_ARG, "gemm: ld_words smaller than ceil(N/32)");
        QNN_REQUIRE(aligned(g.out_bits, 4) && aligned(g.thr, 4), QNN_ERR_ALIGNMENT, "gemm: thr/out_bits must be 4-byte aligned");
    }
    return QNN_OK;
}

static int forced_algo()
{
    const char *e = getenv("QNN_FORCE_ALGO");
    if (!e || !*e) return QNN_ALGO_AUTO;
    if (!strcmp(e, "POPC") || !strcmp(e, "1")) return QNN_ALGO_POPC;
    if (!strcmp(e, "TC_I8") || !strcmp(e, "2")) return QNN_ALGO_TC_I8;
    if (!strcmp(e, "B1_MMA") || !strcmp(e, "3")) return QNN_ALGO_B1_MMA;
    return QNN_ALGO_AUTO;
}

int run_gemm(const GemmArgs &g, int algo, void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (int rc = validate_gemm(g)) return rc;
    QNN_REQUIRE(algo >= QNN_ALGO_AUTO && algo <= QNN_ALGO_B1_MMA, QNN_ERR_INVALID_ARG, "gemm: unknown algo %d", algo);
    if (g.M == 0 || g.N == 0) return QNN_OK;
    if (algo == QNN_ALGO_AUTO) {
        algo = forced_algo();
        if (algo == QNN_ALGO_AUTO) algo = qnn_select_algo(g.M, g.N, g.K, g.ka, g.kb, g.a_mode, g.b_mode);
        // AUTO never fails for want of a workspace: fall back to the CUDA-core path
        if (algo == QNN_ALGO_TC_I8 &&
            (!gemm_tc_supported(g) || ws == nullptr || ws_bytes < gemm_tc_workspace_bytes(g.M, g.N, g.K, g.ka, g.kb)))
            algo = QNN_ALGO_POPC;
        if (algo == QNN_ALGO_B1_MMA && !(g.ka == 1 && g.kb == 1)) algo = QNN_ALGO_POPC;
    }
    switch (algo) {
        case QNN_ALGO_POPC: return launch_gemm_popc(g, st);
        case QNN_ALGO_B1_MMA: return launch_gemm_b1mma(g, st);
        case QNN_ALGO_TC_I8: return launch_gemm_tc(g, ws, ws_bytes, st);
    }
    return fail(QNN_ERR_INVALID_ARG, "gemm: unknown algo");
}

}  // namespace qnn

using namespace qnn;

extern "C" {

int qnn_xnor_gemm(const uint32_t *a, int64_t lda, const uint32_t *b, int64_t ldb, int64_t M, int64_t N, int64_t K,
                  int32_t *out, int64_t ldo, int algo, void *ws, size_t ws_bytes, void *stream)
{
    GemmArgs g{};
    g.a = a; g.b = b; g.lda = lda; g.ldb = ldb; g.ka = g.kb = 1; g.a_mode = g.b_mode = QNN_MODE_PM1;
    g.M = M; g.N = N; g.K = K; g.epilogue = EPI_ROWMAJOR; g.out = out; g.ldo = ldo;
    QNN_REQUIRE(out != nullptr || M == 0 || N == 0, QNN_ERR_INVALID_ARG, "qnn_xnor_gemm: out is NULL");
    return run_gemm(g, algo, ws, ws_bytes, as_stream(stream));
}

int qnn_xnor_gemm_threshold(const uint32_t *a, int64_t lda, const uint32_t *b, int64_t ldb, int64_t M, int64_t N,
                            int64_t K, const int32_t *thr, const uint8_t *flip, uint32_t *out_bits, int64_t ld_words,
                            int algo, void *ws, size_t ws_bytes, void *stream)
{
    GemmArgs g{};
    g.a = a; g.b = b; g.lda = lda; g.ldb = ldb; g.ka = g.kb = 1; g.a_mode = g.b_mode = QNN_MODE_PM1;
    g.M = M; g.N = N; g.K = K; g.epilogue = EPI_BITS; g.thr = thr; g.flip = flip; g.out_bits = out_bits;
    g.ld_bits = ld_words;
    QNN_REQUIRE(out_bits != nullptr || M == 0 || N == 0, QNN_ERR_INVALID_ARG, "qnn_xnor_gemm_threshold: out_bits is NULL");
    return run_gemm(g, algo, ws, ws_bytes, as_stream(stream));
}

int qnn_bitplane_gemm(const uint32_t *a, int ka, int a_mode, int64_t lda, int64_t a_plane_stride, const uint32_t *b,
                      int kb, int b_mode, int64_t ldb, int64_t b_plane_stride, int64_t M, int64_t N, int64_t K,
                      int32_t *out, int64_t ldo, int algo, void *ws, size_t ws_bytes, void *stream)
{
    GemmArgs g{};
    g.a = a; g.b = b; g.lda = lda; g.ldb = ldb; g.ka = ka; g.kb = kb; g.a_mode = a_mode; g.b_mode = b_mode;
    g.a_plane_stride = a_plane_stride; g.b_plane_stride = b_plane_stride;
    g.M = M; g.N = N; g.K = K; g.epilogue = EPI_ROWMAJOR; g.out = out; g.ldo = ldo;
    QNN_REQUIRE(out != nullptr || M == 0 || N == 0, QNN_ERR_INVALID_ARG, "qnn_bitplane_gemm: out is NULL");
    return run_gemm(g, algo, ws, ws_bytes, as_stream(stream));
}

int qnn_bitplane_gemm_threshold(const uint32_t *a, int ka, int a_mode, int64_t lda, int64_t a_plane_stride,
                                const uint32_t *b, int kb, int b_mode, int64_t ldb, int64_t b_plane_stride, int64_t M,
                                int64_t N, int64_t K, const int32_t *thr, const uint8_t *flip, uint32_t *out_bits,
                                int64_t ld_words, int algo, void *ws, size_t ws_bytes, void *stream)
{
    GemmArgs g{};
    g.a = a; g.b = b; g.lda = lda; g.ldb = ldb; g.ka = ka; g.kb = kb; g.a_mode = a_mode; g.b_mode = b_mode;
    g.a_plane_stride = a_plane_stride; g.b_plane_stride = b_plane_stride;
    g.M = M; g.N = N; g.K = K; g.epilogue = EPI_BITS; g.thr = thr; g.flip = flip; g.out_bits = out_bits;
    g.ld_bits = ld_words;
    QNN_REQUIRE(out_bits != nullptr || M == 0 || N == 0, QNN_ERR_INVALID_ARG,
                "qnn_bitplane_gemm_threshold: out_bits is NULL");
    return run_gemm(g, algo, ws, ws_bytes, as_stream(stream));
}

int qnn_select_algo(int64_t M, int64_t N, int64_t K, int ka, int kb, int a_mode, int b_mode)
{
    // Measured on B200: the 1-bit mma.sync path never beats xor+popc on the CUDA cores, so it is never picked.
    // The tcgen05 int8 path costs one pass whatever the plane counts and overtakes the CUDA-core path once the
    // equivalent plane-pair work M*N*K*ka*kb reaches about 2^31; below that its expansion passes and launch
    // latencies dominate.
    if (M <= 0 || N <= 0 || K <= 0) return QNN_ALGO_POPC;
    if ((a_mode == QNN_MODE_PM1 && ka > 7) || (b_mode == QNN_MODE_PM1 && kb > 7)) return QNN_ALGO_POPC;
    const double work = (double)M * (double)N * (double)K * (double)ka * (double)kb;
    return work >= 2147483648.0 ? QNN_ALGO_TC_I8 : QNN_ALGO_POPC;
}

size_t qnn_workspace_bytes(int op, int64_t M, int64_t N, int64_t K, int ka, int kb, int algo)
{
    if (M <= 0 || N <= 0 || K <= 0) return 0;
    size_t bytes = 0;
    if (op == QNN_OP_CONV2D) {
        bytes += round_up(sizeof(uint32_t) * (size_t)M * (size_t)ceil_div(K, 32), 256);   // packed im2col
        ka = kb = 1;
    }
    if (algo == QNN_ALGO_TC_I8 || algo == QNN_ALGO_AUTO) bytes += gemm_tc_workspace_bytes(M, N, K, ka, kb);
    return bytes;
}

}  // extern "C"
