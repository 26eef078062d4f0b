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
    QNN_REQUIRE(g.out != nullptr || g.out_bits != nullptr || g.out_form != nullptr, QNN_ERR_INVALID_ARG,
                "gemm: no output buffer");
    if (g.K > 0) {
        // an operand is given as packed planes, or already in a tensor-core form
        QNN_REQUIRE((g.a || g.a_tc) && (g.b || g.b_tc), QNN_ERR_INVALID_ARG, "gemm: NULL operand");
        if (!g.a_tc) {
            QNN_REQUIRE(g.lda >= kw, QNN_ERR_INVALID_ARG, "gemm: lda smaller than ceil(K/32)");
            QNN_REQUIRE(g.ka == 1 || g.a_plane_stride >= g.M * g.lda, QNN_ERR_INVALID_ARG, "gemm: a_plane_stride too small");
            QNN_REQUIRE(aligned(g.a, 4), QNN_ERR_ALIGNMENT, "gemm: operands must be 4-byte aligned");
        }
        if (!g.b_tc) {
            QNN_REQUIRE(g.ldb >= kw, QNN_ERR_INVALID_ARG, "gemm: ldb smaller than ceil(K/32)");
            QNN_REQUIRE(g.kb == 1 || g.b_plane_stride >= g.N * g.ldb, QNN_ERR_INVALID_ARG, "gemm: b_plane_stride too small");
            QNN_REQUIRE(aligned(g.b, 4), QNN_ERR_ALIGNMENT, "gemm: operands must be 4-byte aligned");
        }
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
    if (!strcmp(e, "TC_FP4") || !strcmp(e, "4")) return QNN_ALGO_TC_FP4;
    if (!strcmp(e, "B1_MMA") || !strcmp(e, "3")) return QNN_ALGO_B1_MMA;
    return QNN_ALGO_AUTO;
}

int run_gemm(const GemmArgs &g, int algo, void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (int rc = validate_gemm(g)) return rc;
    QNN_REQUIRE(algo >= QNN_ALGO_AUTO && algo <= QNN_ALGO_TC_PACKED, QNN_ERR_INVALID_ARG, "gemm: unknown algo %d", algo);
    if (g.M == 0 || g.N == 0) return QNN_OK;
    if (algo == QNN_ALGO_AUTO) {
        algo = forced_algo();
        if (algo == QNN_ALGO_AUTO) algo = qnn_select_algo(g.M, g.N, g.K, g.ka, g.kb, g.a_mode, g.b_mode);
        if (algo == QNN_ALGO_TC_PACKED && !gemm_smallm_supported(g)) algo = QNN_ALGO_TC_FP4;      // (prepared operands, unaligned rows, ...)
        // AUTO never fails for want of a workspace or of a fitting form: fall back to the CUDA-core path
        if (algo == QNN_ALGO_TC_I8 || algo == QNN_ALGO_TC_FP4) {
            const int form = algo == QNN_ALGO_TC_FP4 ? QNN_FORM_FP4 : QNN_FORM_I8;
            const bool fits = tc_form_holds(form, g.ka, g.a_mode) && tc_form_holds(form, g.kb, g.b_mode) &&
                              (form != QNN_FORM_FP4 || tc_pick_form(g.ka, g.a_mode, g.kb, g.b_mode, g.K) == QNN_FORM_FP4);
            const int64_t kw = g.kwords > 0 ? g.kwords : ceil_div(g.K, 32);
            const size_t need = (g.a_tc ? 0 : round_up((size_t)g.M * (size_t)tc_row_pitch(kw, form), 256)) +
                                (g.b_tc ? 0 : round_up((size_t)g.N * (size_t)tc_row_pitch(kw, form), 256));
            if (!fits || kw == 0) {
                algo = QNN_ALGO_POPC;
            } else if (need > 0 && (ws == nullptr || !aligned(ws, 256) || ws_bytes < need)) {
                // The result is the same, the speed is not: leave word of it where the caller can find it.  Small batches
                // still run on the tensor cores, straight from the packed planes; the rest on the CUDA cores.
                const bool packed_ok = g.M <= 1024 && gemm_smallm_supported(g);
                note("gemm: QNN_ALGO_AUTO ran the %s instead of the tensor-core kernel on rewritten operands: that one needs a "
                     "256-byte aligned workspace of %zu bytes (got %zu at %p)",
                     packed_ok ? "tensor-core kernel on packed tiles" : "CUDA-core kernel", need, ws_bytes, ws);
                algo = packed_ok ? QNN_ALGO_TC_PACKED : QNN_ALGO_POPC;
            }
        }
        if (algo == QNN_ALGO_B1_MMA && !(g.ka == 1 && g.kb == 1)) algo = QNN_ALGO_POPC;
    }
    if (algo == QNN_ALGO_TC_PACKED) return launch_gemm_smallm(g, st);
    if (algo == QNN_ALGO_POPC || algo == QNN_ALGO_B1_MMA)
        QNN_REQUIRE(g.a && g.b && !g.out_form, QNN_ERR_INVALID_ARG, "gemm: the CUDA-core paths take packed planes and write no form output");
    switch (algo) {
        case QNN_ALGO_POPC: return launch_gemm_popc(g, st);
        case QNN_ALGO_B1_MMA: return launch_gemm_b1mma(g, st);
        case QNN_ALGO_TC_I8: return launch_gemm_tc(g, QNN_FORM_I8, ws, ws_bytes, st);
        case QNN_ALGO_TC_FP4: return launch_gemm_tc(g, QNN_FORM_FP4, ws, ws_bytes, st);
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

int qnn_tc_form(int ka, int a_mode, int kb, int b_mode, int64_t K)
{
    if (ka < 1 || ka > 8 || kb < 1 || kb > 8 || K < 0) return 0;
    return tc_pick_form(ka, a_mode, kb, b_mode, K);
}

int64_t qnn_tc_row_bytes(int64_t K, int form)
{
    if (K < 0 || (form != QNN_FORM_I8 && form != QNN_FORM_FP4)) return 0;
    return tc_row_pitch(ceil_div(K, 32), form);
}

size_t qnn_tc_operand_bytes(int64_t rows, int64_t K, int form)
{
    if (rows <= 0) return 0;
    return (size_t)rows * (size_t)qnn_tc_row_bytes(K, form);
}

int qnn_tc_prepack(const uint32_t *planes, int nplanes, int mode, int64_t ld, int64_t plane_stride, int64_t rows,
                   int64_t K, int form, void *out, int64_t ld_bytes, void *stream)
{
    QNN_REQUIRE(rows >= 0 && K >= 0, QNN_ERR_INVALID_ARG, "qnn_tc_prepack: negative size");
    QNN_REQUIRE(nplanes >= 1 && nplanes <= 8 && (mode == QNN_MODE_U01 || mode == QNN_MODE_PM1), QNN_ERR_INVALID_ARG,
                "qnn_tc_prepack: bad plane count or mode");
    QNN_REQUIRE(form == QNN_FORM_I8 || form == QNN_FORM_FP4, QNN_ERR_INVALID_ARG, "qnn_tc_prepack: unknown form %d", form);
    QNN_REQUIRE(tc_form_holds(form, nplanes, mode), QNN_ERR_UNSUPPORTED,
                "qnn_tc_prepack: values of %d planes do not fit form %d", nplanes, form);
    if (rows == 0 || K == 0) return QNN_OK;
    const int64_t kwords = ceil_div(K, 32);
    QNN_REQUIRE(planes && out, QNN_ERR_INVALID_ARG, "qnn_tc_prepack: NULL pointer");
    QNN_REQUIRE(ld >= kwords && (nplanes == 1 || plane_stride >= rows * ld), QNN_ERR_INVALID_ARG,
                "qnn_tc_prepack: ld or plane stride too small");
    QNN_REQUIRE(aligned(out, 16) && ld_bytes % 16 == 0 && ld_bytes >= tc_row_bytes(kwords, form), QNN_ERR_ALIGNMENT,
                "qnn_tc_prepack: out needs a 16-byte aligned base and a row stride that is a multiple of 16 covering K");
    return tc_expand(planes, nplanes, mode, ld, plane_stride, rows, kwords, kwords, (int)(K - 32 * (kwords - 1)), form,
                     static_cast<uint8_t *>(out), ld_bytes, as_stream(stream));
}

int qnn_tc_gemm(const qnn_tc_operand *a, const qnn_tc_operand *b, int64_t M, int64_t N, int64_t K, const qnn_tc_output *o,
                void *stream)
{
    QNN_REQUIRE(a && b && o, QNN_ERR_INVALID_ARG, "qnn_tc_gemm: NULL descriptor");
    QNN_REQUIRE(a->form == b->form, QNN_ERR_INVALID_ARG, "qnn_tc_gemm: operands are in different forms");
    GemmArgs g{};
    g.ka = a->planes; g.kb = b->planes; g.a_mode = a->mode; g.b_mode = b->mode;
    g.M = M; g.N = N; g.K = K;
    g.a_tc = a->data; g.a_tc_form = a->form; g.a_tc_ld = a->ld_bytes;
    g.b_tc = b->data; g.b_tc_form = b->form; g.b_tc_ld = b->ld_bytes;
    g.epilogue = o->out ? EPI_ROWMAJOR : EPI_BITS;
    g.out = o->out; g.ldo = o->ldo; g.thr = o->thr; g.flip = o->flip; g.out_bits = o->out_bits; g.ld_bits = o->ld_words;
    g.out_form = o->out_form; g.out_form_kind = o->out_form_kind; g.ld_form = o->ld_form_bytes;
    QNN_REQUIRE(M >= 0 && N >= 0 && K >= 1, QNN_ERR_INVALID_ARG, "qnn_tc_gemm: bad size");
    QNN_REQUIRE(K < (int64_t)1 << 31, QNN_ERR_INVALID_ARG, "qnn_tc_gemm: K must be below 2^31");
    QNN_REQUIRE(g.ka >= 1 && g.ka <= 8 && g.kb >= 1 && g.kb <= 8, QNN_ERR_INVALID_ARG, "qnn_tc_gemm: plane counts must be in 1..8");
    const int64_t la = (1 << g.ka) - 1, lb = (1 << g.kb) - 1;
    QNN_REQUIRE(la * lb <= (((int64_t)1 << 31) - 1) / K, QNN_ERR_OVERFLOW, "qnn_tc_gemm: result may not fit int32");
    if (M == 0 || N == 0) return QNN_OK;
    QNN_REQUIRE(a->data && b->data, QNN_ERR_INVALID_ARG, "qnn_tc_gemm: NULL operand");
    QNN_REQUIRE(o->out || o->out_bits || o->out_form, QNN_ERR_INVALID_ARG, "qnn_tc_gemm: no output buffer");
    QNN_REQUIRE(!o->out || o->ldo >= N, QNN_ERR_INVALID_ARG, "qnn_tc_gemm: ldo smaller than N");
    QNN_REQUIRE(!(o->out_bits || o->out_form) || o->thr, QNN_ERR_INVALID_ARG, "qnn_tc_gemm: thresholds required");
    QNN_REQUIRE(!o->out_bits || o->ld_words >= ceil_div(N, 32), QNN_ERR_INVALID_ARG, "qnn_tc_gemm: ld_words too small");
    const int64_t rb = tc_row_bytes(ceil_div(K, 32), a->form);
    // A in the int8 form may be a plain byte matrix whose rows are only K bytes apart: the rest of the last word reads 0
    const int64_t a_min = a->form == QNN_FORM_I8 ? K : rb;
    QNN_REQUIRE(a->ld_bytes >= a_min && b->ld_bytes >= rb, QNN_ERR_INVALID_ARG, "qnn_tc_gemm: operand row stride smaller than K needs");
    return launch_gemm_tc(g, a->form, nullptr, 0, as_stream(stream));
}

int qnn_select_algo(int64_t M, int64_t N, int64_t K, int ka, int kb, int a_mode, int b_mode)
{
    // Measured on B200 (whole call from packed planes, L2 flushed; see the bench's `algorithms` block):
    //  - the 1-bit mma.sync path never beats xor+popc on the CUDA cores, so it is never picked;
    //  - a tensor-core path costs one pass whatever the plane counts and overtakes the CUDA-core path once the
    //    equivalent plane-pair work M*N*K*ka*kb reaches about 2 * 10^7 (128 x 512 x 2048: 15.4 us against 19.4 us;
    //    64 x 256 x 1024: 11.3 us against 13.3 us; below that every path is one launch of 11-13 us);
    //  - the kernel that expands packed tiles itself (one launch, no operand rewriting) wins while its 128 x 32 tiles
    //    fit one wave of CTAs and K is short (512 x 1024 x 2048: 14.3 us against 15.4 us; at K = 4096 the two are level,
    //    beyond one wave it re-expands too much: 1024^3 18.4 us against 13.5 us).
    // The answer assumes operands the chosen kernel accepts (alignment, a workspace for the rewritten operands);
    // QNN_ALGO_AUTO falls back at call time where they are not.
    if (M <= 0 || N <= 0 || K <= 0) return QNN_ALGO_POPC;
    const int form = tc_pick_form(ka, a_mode, kb, b_mode, K);
    if (form == 0) return QNN_ALGO_POPC;
    const double work = (double)M * (double)N * (double)K * (double)ka * (double)kb;
    if (work < 16777216.0) return QNN_ALGO_POPC;
    if (form == QNN_FORM_FP4 && ka == 1 && kb == 1 && K <= 2048 && ceil_div(M, 128) * ceil_div(N, 32) <= sm_count())
        return QNN_ALGO_TC_PACKED;
    return form == QNN_FORM_FP4 ? QNN_ALGO_TC_FP4 : QNN_ALGO_TC_I8;
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
    if (algo == QNN_ALGO_TC_FP4) {
        const int64_t rb = tc_row_pitch(ceil_div(K, 32), QNN_FORM_FP4);
        bytes += round_up((size_t)M * (size_t)rb, 256) + round_up((size_t)N * (size_t)rb, 256);
    }
    return bytes;
}

}  // extern "C"
