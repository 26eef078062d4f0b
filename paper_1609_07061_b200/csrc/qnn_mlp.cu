// Algorithm 4 ("Running a BNN with L layers") as a chain of library calls on
// one stream: bit-plane first layer, thresholded XNOR hidden layers with packed
// activations ping-ponging between two workspace buffers, int32 scores last.
#include "qnn_internal.cuh"

namespace qnn {
namespace {

struct MlpPlan {
    int64_t kw0;            // words per row of one input plane
    size_t off_x, off_scores, off_planes, off_act0, off_act1, off_gemm;
    size_t gemm_bytes, total;
};

int plan_mlp(int64_t M, int in_bits, const qnn_mlp_layer *layers, int L, int algo, int host_io, MlpPlan *p)
{
    QNN_REQUIRE(layers != nullptr && L >= 1, QNN_ERR_INVALID_ARG, "mlp: need at least one layer");
    QNN_REQUIRE(M >= 0 && in_bits >= 1 && in_bits <= 8, QNN_ERR_INVALID_ARG, "mlp: bad batch or input bit-width");
    for (int l = 0; l < L; ++l) {
        QNN_REQUIRE(layers[l].K >= 1 && layers[l].N >= 1 && layers[l].w != nullptr, QNN_ERR_INVALID_ARG,
                    "mlp: layer %d has a bad shape or NULL weights", l);
        QNN_REQUIRE(layers[l].ldw >= ceil_div(layers[l].K, 32), QNN_ERR_INVALID_ARG, "mlp: layer %d ldw too small", l);
        if (l > 0) QNN_REQUIRE(layers[l].K == layers[l - 1].N, QNN_ERR_INVALID_ARG, "mlp: layer %d K != previous N", l);
        if (l < L - 1) QNN_REQUIRE(layers[l].thr != nullptr, QNN_ERR_INVALID_ARG, "mlp: hidden layer %d needs thresholds", l);
    }
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += round_up(bytes > 0 ? bytes : 1, 256); return o; };
    p->kw0 = round_up((size_t)ceil_div(layers[0].K, 32), 4);
    p->off_x = host_io ? take((size_t)M * (size_t)layers[0].K) : 0;
    p->off_scores = host_io ? take(sizeof(int32_t) * (size_t)M * (size_t)layers[L - 1].N) : 0;
    p->off_planes = take(sizeof(uint32_t) * (size_t)in_bits * (size_t)M * (size_t)p->kw0);
    int64_t maxw = 4;
    for (int l = 0; l < L - 1; ++l) {
        const int64_t wds = (int64_t)round_up((size_t)ceil_div(layers[l].N, 32), 4);
        if (wds > maxw) maxw = wds;
    }
    p->off_act0 = take(sizeof(uint32_t) * (size_t)M * (size_t)maxw);
    p->off_act1 = take(sizeof(uint32_t) * (size_t)M * (size_t)maxw);
    size_t gb = 0;
    for (int l = 0; l < L; ++l) {
        const size_t b = qnn_workspace_bytes(l == 0 ? QNN_OP_BITPLANE_GEMM : QNN_OP_XNOR_GEMM, M, layers[l].N,
                                             layers[l].K, l == 0 ? in_bits : 1, 1, algo);
        if (b > gb) gb = b;
    }
    p->gemm_bytes = gb;
    p->off_gemm = take(gb);
    p->total = off;
    return QNN_OK;
}

int run_mlp(const uint8_t *x_dev, int64_t M, int in_bits, const qnn_mlp_layer *layers, int L, int32_t *scores_dev,
            int algo, char *ws, const MlpPlan &p, cudaStream_t st)
{
    if (M == 0) return QNN_OK;
    uint32_t *planes = reinterpret_cast<uint32_t *>(ws + p.off_planes);
    uint32_t *act[2] = {reinterpret_cast<uint32_t *>(ws + p.off_act0), reinterpret_cast<uint32_t *>(ws + p.off_act1)};
    void *gws = ws + p.off_gemm;
    const int64_t plane_stride = M * p.kw0;
    if (int rc = qnn_pack_planes_u8(x_dev, M, layers[0].K, layers[0].K, in_bits, planes, p.kw0, plane_stride, nullptr, st))
        return rc;
    const uint32_t *cur = planes;
    int64_t cur_ld = p.kw0;
    for (int l = 0; l < L; ++l) {
        const qnn_mlp_layer &ly = layers[l];
        const bool last = (l == L - 1);
        GemmArgs g{};
        g.a = cur; g.lda = cur_ld; g.b = ly.w; g.ldb = ly.ldw;
        g.ka = (l == 0) ? in_bits : 1; g.kb = 1;
        g.a_mode = (l == 0) ? QNN_MODE_U01 : QNN_MODE_PM1; g.b_mode = QNN_MODE_PM1;
        g.a_plane_stride = (l == 0) ? plane_stride : 0;
        g.M = M; g.N = ly.N; g.K = ly.K;
        if (last) {
            g.epilogue = EPI_ROWMAJOR; g.out = scores_dev; g.ldo = ly.N;
        } else {
            g.epilogue = EPI_BITS; g.thr = ly.thr; g.flip = ly.flip; g.out_bits = act[l & 1];
            g.ld_bits = (int64_t)round_up((size_t)ceil_div(ly.N, 32), 4);
        }
        if (int rc = run_gemm(g, algo, gws, p.gemm_bytes, st)) return rc;
        if (!last) { cur = act[l & 1]; cur_ld = g.ld_bits; }
    }
    return QNN_OK;
}

}  // namespace
}  // namespace qnn

using namespace qnn;

extern "C" {

size_t qnn_mlp_workspace_bytes(int64_t M, int in_bits, const qnn_mlp_layer *layers, int L, int algo, int host_io)
{
    MlpPlan p;
    if (plan_mlp(M, in_bits, layers, L, algo, host_io, &p) != QNN_OK) return 0;
    return p.total;
}

int qnn_mlp_forward(const uint8_t *x, int64_t M, int in_bits, const qnn_mlp_layer *layers, int L, int32_t *scores,
                    int algo, void *ws, size_t ws_bytes, void *stream)
{
    MlpPlan p;
    if (int rc = plan_mlp(M, in_bits, layers, L, algo, 0, &p)) return rc;
    if (M == 0) return QNN_OK;
    QNN_REQUIRE(x && scores, QNN_ERR_INVALID_ARG, "qnn_mlp_forward: NULL input or output");
    QNN_REQUIRE(ws && aligned(ws, 256) && ws_bytes >= p.total, QNN_ERR_WORKSPACE,
                "qnn_mlp_forward: workspace of at least %zu bytes (256-byte aligned) required", p.total);
    return run_mlp(x, M, in_bits, layers, L, scores, algo, static_cast<char *>(ws), p, as_stream(stream));
}

int qnn_mlp_forward_host(const uint8_t *x_host, int64_t M, int in_bits, const qnn_mlp_layer *layers, int L,
                         int32_t *scores_host, int algo, void *ws, size_t ws_bytes, void *stream)
{
    MlpPlan p;
    if (int rc = plan_mlp(M, in_bits, layers, L, algo, 1, &p)) return rc;
    if (M == 0) return QNN_OK;
    QNN_REQUIRE(x_host && scores_host, QNN_ERR_INVALID_ARG, "qnn_mlp_forward_host: NULL input or output");
    QNN_REQUIRE(ws && aligned(ws, 256) && ws_bytes >= p.total, QNN_ERR_WORKSPACE,
                "qnn_mlp_forward_host: workspace of at least %zu bytes (256-byte aligned) required", p.total);
    cudaStream_t st = as_stream(stream);
    char *base = static_cast<char *>(ws);
    uint8_t *x_dev = reinterpret_cast<uint8_t *>(base + p.off_x);
    int32_t *s_dev = reinterpret_cast<int32_t *>(base + p.off_scores);
    const size_t in_bytes = (size_t)M * (size_t)layers[0].K;
    const size_t out_bytes = sizeof(int32_t) * (size_t)M * (size_t)layers[L - 1].N;
    QNN_CUDA(cudaMemcpyAsync(x_dev, x_host, in_bytes, cudaMemcpyHostToDevice, st));
    if (int rc = run_mlp(x_dev, M, in_bits, layers, L, s_dev, algo, base, p, st)) return rc;
    QNN_CUDA(cudaMemcpyAsync(scores_host, s_dev, out_bytes, cudaMemcpyDeviceToHost, st));
    QNN_CUDA(cudaStreamSynchronize(st));
    return QNN_OK;
}

}  // extern "C"
