// Algorithm 4 ("Running a BNN with L layers") as a chain of library calls on
// one stream: bit-plane first layer, thresholded XNOR hidden layers with packed
// activations ping-ponging between two workspace buffers, int32 scores last.
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include "qnn_internal.cuh"

namespace qnn {
namespace {

struct LayerChoice {
    int algo;               // resolved algorithm of this layer (never AUTO)
    int form;               // tensor-core form when algo is a tensor-core one, else 0
};

struct MlpPlan {
    int64_t kw0;            // words per row of one input plane
    size_t off_x, off_scores, off_planes, off_act0, off_act1, off_gemm;
    size_t gemm_bytes, act_bytes, total;
};

inline bool is_tc(int algo) { return algo == QNN_ALGO_TC_I8 || algo == QNN_ALGO_TC_FP4; }

// Copies a dense byte matrix [rows, K] (K a multiple of 16) to rows `pitch` bytes apart.  The tensor-core
// product reads its operands in 128-byte boxes; rows that start on 128-byte lines halve the lines a box touches.
__global__ void __launch_bounds__(256) repitch_rows_kernel(const uint4 *__restrict__ src, int64_t rows, int64_t k16,
                                                           uint4 *__restrict__ dst, int64_t pitch16)
{
    griddep_launch_dependents();
    griddep_wait();
    const int64_t total = rows * k16;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = e / k16, c = e - r * k16;
        dst[r * pitch16 + c] = __ldcs(src + e);
    }
}

int resolve_env_algo()
{
    const char *e = getenv("QNN_FORCE_ALGO");
    if (!e || !*e) return QNN_ALGO_AUTO;
    if (!strcmp(e, "POPC") || !strcmp(e, "1")) return QNN_ALGO_POPC;
    if (!strcmp(e, "TC_I8") || !strcmp(e, "2")) return QNN_ALGO_TC_I8;
    if (!strcmp(e, "B1_MMA") || !strcmp(e, "3")) return QNN_ALGO_B1_MMA;
    if (!strcmp(e, "TC_FP4") || !strcmp(e, "4")) return QNN_ALGO_TC_FP4;
    if (!strcmp(e, "TC_PACKED") || !strcmp(e, "5")) return QNN_ALGO_TC_PACKED;
    return QNN_ALGO_AUTO;
}

// Algorithm and form of layer l.  A forced algorithm that cannot run a layer's operands (the 1-bit
// paths on the 8-plane first layer, a form that does not hold the values) falls back to the one
// AUTO would take, so that a network always runs.
LayerChoice choose_layer(int64_t M, int in_bits, const qnn_mlp_layer *layers, int l, int algo)
{
    const qnn_mlp_layer &ly = layers[l];
    const int ka = l == 0 ? in_bits : 1;
    const int a_mode = l == 0 ? QNN_MODE_U01 : QNN_MODE_PM1;
    const int best_form = tc_pick_form(ka, a_mode, 1, QNN_MODE_PM1, ly.K);
    if (algo == QNN_ALGO_AUTO) algo = resolve_env_algo();
    LayerChoice c{algo, 0};
    if (algo == QNN_ALGO_AUTO) {
        c.algo = qnn_select_algo(M, ly.N, ly.K, ka, 1, a_mode, QNN_MODE_PM1);
        // (inside a network the layers hand their activations over in tensor-core form and the weights may be prepared:
        // the packed-tile kernel, which takes packed planes only, is left to single products)
        if (c.algo == QNN_ALGO_TC_PACKED) c.algo = QNN_ALGO_TC_FP4;
    }
    if (c.algo == QNN_ALGO_B1_MMA && ka != 1) c.algo = QNN_ALGO_POPC;
    if (c.algo == QNN_ALGO_TC_PACKED && best_form != QNN_FORM_FP4) c.algo = QNN_ALGO_POPC;     // (more than two planes, or sums beyond 2^24)
    if (c.algo == QNN_ALGO_TC_FP4 && best_form != QNN_FORM_FP4) c.algo = best_form ? QNN_ALGO_TC_I8 : QNN_ALGO_POPC;
    if (c.algo == QNN_ALGO_TC_I8 && !(tc_form_holds(QNN_FORM_I8, ka, a_mode))) c.algo = QNN_ALGO_POPC;
    if (c.algo == QNN_ALGO_TC_FP4) c.form = QNN_FORM_FP4;
    if (c.algo == QNN_ALGO_TC_I8) c.form = QNN_FORM_I8;
    return c;
}

int plan_mlp(int64_t M, int in_bits, const qnn_mlp_layer *layers, int L, int algo, int host_io, MlpPlan *p)
{
    QNN_REQUIRE(layers != nullptr && L >= 1, QNN_ERR_INVALID_ARG, "mlp: need at least one layer");
    QNN_REQUIRE(M >= 0 && in_bits >= 1 && in_bits <= 8, QNN_ERR_INVALID_ARG, "mlp: bad batch or input bit-width");
    QNN_REQUIRE(algo >= QNN_ALGO_AUTO && algo <= QNN_ALGO_TC_PACKED, QNN_ERR_INVALID_ARG, "mlp: unknown algo %d", algo);
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
    // an activation buffer holds one hidden layer's output either as packed bits or in a tensor-core form
    int64_t max_row = 16;
    for (int l = 0; l < L - 1; ++l) {
        const int64_t wds = (int64_t)round_up((size_t)ceil_div(layers[l].N, 32), 4);
        const int64_t row = wds * 32;                      // the int8 form is the widest: one byte per element
        if (row > max_row) max_row = row;
    }
    p->act_bytes = (size_t)M * (size_t)max_row;
    // each buffer holds a layer's packed bits (first quarter at most) and its tensor-core form side by side
    p->off_act0 = take(p->act_bytes + (p->act_bytes >> 2));
    p->off_act1 = take(p->act_bytes + (p->act_bytes >> 2));
    size_t gb = 0;
    for (int l = 0; l < L; ++l) {
        const size_t b = qnn_workspace_bytes(l == 0 ? QNN_OP_BITPLANE_GEMM : QNN_OP_XNOR_GEMM, M, layers[l].N,
                                             layers[l].K, l == 0 ? in_bits : 1, 1, QNN_ALGO_AUTO);
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
    char *act[2] = {ws + p.off_act0, ws + p.off_act1};
    void *gws = ws + p.off_gemm;
    const int64_t plane_stride = M * p.kw0;

    LayerChoice choice[64];
    QNN_REQUIRE(L <= 64, QNN_ERR_UNSUPPORTED, "mlp: at most 64 layers");
    for (int l = 0; l < L; ++l) choice[l] = choose_layer(M, in_bits, layers, l, algo);
    // A few-unit last layer is too little work for the tensor cores to win when its operands have to be rewritten
    // first; with weights already in form and the previous layer able to hand its signs over in form there is nothing
    // to rewrite, and the tensor-core kernel is the faster one (measured: 10000 x 10 x 4096 head, step 176 -> 173 us).
    if (algo == QNN_ALGO_AUTO && resolve_env_algo() == QNN_ALGO_AUTO && L >= 2 && choice[L - 1].algo == QNN_ALGO_POPC &&
        is_tc(choice[L - 2].algo) && M >= 1024) {
        const qnn_mlp_layer &ly = layers[L - 1];
        const int form = tc_pick_form(1, QNN_MODE_PM1, 1, QNN_MODE_PM1, ly.K);
        if (form != 0 && ly.w_tc != nullptr && ly.w_tc_form == form) {
            choice[L - 1].algo = form == QNN_FORM_FP4 ? QNN_ALGO_TC_FP4 : QNN_ALGO_TC_I8;
            choice[L - 1].form = form;
        }
    }

    // what the previous layer left behind for this one
    const uint32_t *cur_bits = nullptr; int64_t cur_ld = 0;
    const void *cur_form = nullptr; int cur_form_kind = 0; int64_t cur_form_ld = 0;

    for (int l = 0; l < L; ++l) {
        const qnn_mlp_layer &ly = layers[l];
        const LayerChoice &c = choice[l];
        const bool last = (l == L - 1);
        GemmArgs g{};
        g.b = ly.w; g.ldb = ly.ldw; g.kb = 1; g.b_mode = QNN_MODE_PM1;
        g.ka = (l == 0) ? in_bits : 1;
        g.a_mode = (l == 0) ? QNN_MODE_U01 : QNN_MODE_PM1;
        g.M = M; g.N = ly.N; g.K = ly.K;
        if (l == 0) {
            // 8-bit inputs ARE the int8-form operand (Eq. 8 recomposed): no plane split, no expansion
            const bool direct = c.form == QNN_FORM_I8 && in_bits == 8 && (ly.K % 16 == 0) && aligned(x_dev, 16);
            if (direct) {
                g.a_tc = x_dev; g.a_tc_form = QNN_FORM_I8; g.a_tc_ld = ly.K;
                if (ly.K % 128 != 0) {
                    // rows of the input re-spaced to whole 128-byte lines (the plane buffer is free on this path)
                    const int64_t pitch = p.kw0 * 32;
                    const int64_t total = M * (ly.K / 16);
                    const int64_t need = ceil_div(total, 256), cap = (int64_t)sm_count() * 16;
                    QNN_CUDA(launch_pdl(repitch_rows_kernel, dim3((unsigned)(need < cap ? need : cap)), dim3(256), 0, st,
                                        reinterpret_cast<const uint4 *>(x_dev), M, ly.K / 16, reinterpret_cast<uint4 *>(planes), pitch / 16));
                    if (int rc = check_launch("mlp input re-spacing")) return rc;
                    g.a_tc = planes; g.a_tc_ld = pitch;
                }
            } else {
                if (int rc = qnn_pack_planes_u8(x_dev, M, ly.K, ly.K, in_bits, planes, p.kw0, plane_stride, nullptr, st))
                    return rc;
                g.a = planes; g.lda = p.kw0; g.a_plane_stride = plane_stride;
            }
        } else if (cur_form != nullptr && cur_form_kind == c.form) {
            g.a_tc = cur_form; g.a_tc_form = cur_form_kind; g.a_tc_ld = cur_form_ld;
        } else {
            g.a = cur_bits; g.lda = cur_ld;
        }
        if (is_tc(c.algo) && ly.w_tc != nullptr && ly.w_tc_form == c.form) {
            g.b_tc = ly.w_tc; g.b_tc_form = ly.w_tc_form; g.b_tc_ld = ly.w_tc_ld;
        }
        if (last) {
            g.epilogue = EPI_ROWMAJOR; g.out = scores_dev; g.ldo = ly.N;
        } else {
            // hand the next layer what it consumes: its tensor-core form when this layer can write it, else packed bits
            const LayerChoice &nx = choice[l + 1];
            char *buf = act[l & 1];
            const int64_t wds = (int64_t)round_up((size_t)ceil_div(ly.N, 32), 4);
            g.epilogue = EPI_BITS; g.thr = ly.thr; g.flip = ly.flip;
            const bool give_form = is_tc(c.algo) && is_tc(nx.algo);
            cur_bits = nullptr; cur_form = nullptr;
            if (give_form) {
                g.out_form = buf + (p.act_bytes >> 2); g.out_form_kind = nx.form; g.ld_form = tc_row_pitch(wds, nx.form);
                cur_form = g.out_form; cur_form_kind = nx.form; cur_form_ld = g.ld_form;
            } else {
                g.out_bits = reinterpret_cast<uint32_t *>(buf); g.ld_bits = wds;
                cur_bits = g.out_bits; cur_ld = wds;
            }
        }
        if (int rc = run_gemm(g, c.algo, gws, p.gemm_bytes, st)) return rc;
    }
    return QNN_OK;
}

// One non-blocking stream per device for the host entry point's input copies, created on first use and kept.
cudaStream_t copy_stream()
{
    static std::mutex mu;
    static cudaStream_t streams[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (streams[dev] == nullptr && cudaStreamCreateWithFlags(&streams[dev], cudaStreamNonBlocking) != cudaSuccess) {
        (void)cudaGetLastError();
        streams[dev] = nullptr;
    }
    return streams[dev];
}

}  // namespace
}  // namespace qnn

namespace qnn {
namespace {

// One pass from host buffers, queued on `st` (and on the library's copy stream for the overlapped input chunks):
// input copies, the layers chunk by chunk, the copy of the scores back.  Does not synchronise.  Also runs under
// stream capture: the copy stream is forked from `st` by an event and joined back by the chunks' events.
int issue_host_pass(const uint8_t *x_host, int64_t M, int in_bits, const qnn_mlp_layer *layers, int L, int32_t *scores_host,
                    int algo, char *base, const MlpPlan &p, int chunks, cudaStream_t st)
{
    uint8_t *x_dev = reinterpret_cast<uint8_t *>(base + p.off_x);
    int32_t *s_dev = reinterpret_cast<int32_t *>(base + p.off_scores);
    const int64_t K0 = layers[0].K, NL = layers[L - 1].N;
    if (chunks > 8) chunks = 8;
    cudaStream_t cs = chunks > 1 ? copy_stream() : nullptr;
    if (chunks == 1 || cs == nullptr) {
        QNN_CUDA(cudaMemcpyAsync(x_dev, x_host, (size_t)M * (size_t)K0, cudaMemcpyHostToDevice, st));
        if (int rc = run_mlp(x_dev, M, in_bits, layers, L, s_dev, algo, base, p, st)) return rc;
    } else {
        const int64_t rows_c = (int64_t)round_up((size_t)ceil_div(M, chunks), 256);   // whole 256-row tiles per chunk
        cudaEvent_t ev[9] = {};
        int rc = QNN_OK;
        for (int c = 0; c <= chunks && rc == QNN_OK; ++c)
            if (cudaEventCreateWithFlags(&ev[c], cudaEventDisableTiming) != cudaSuccess) rc = fail(QNN_ERR_CUDA, "qnn_mlp_forward_host: cudaEventCreate failed");
        if (rc == QNN_OK) {
            // the copies start after whatever the caller already queued on its stream
            if (cudaEventRecord(ev[chunks], st) != cudaSuccess || cudaStreamWaitEvent(cs, ev[chunks], 0) != cudaSuccess)
                rc = fail(QNN_ERR_CUDA, "qnn_mlp_forward_host: stream ordering failed");
        }
        for (int c = 0; c < chunks && rc == QNN_OK; ++c) {
            const int64_t r0 = c * rows_c, rows = (r0 + rows_c <= M ? rows_c : M - r0);
            if (rows <= 0) break;
            if (cudaMemcpyAsync(x_dev + r0 * K0, x_host + r0 * K0, (size_t)rows * (size_t)K0, cudaMemcpyHostToDevice, cs) != cudaSuccess ||
                cudaEventRecord(ev[c], cs) != cudaSuccess)
                rc = fail(QNN_ERR_CUDA, "qnn_mlp_forward_host: chunk copy failed");
        }
        for (int c = 0; c < chunks && rc == QNN_OK; ++c) {
            const int64_t r0 = c * rows_c, rows = (r0 + rows_c <= M ? rows_c : M - r0);
            if (rows <= 0) break;
            if (cudaStreamWaitEvent(st, ev[c], 0) != cudaSuccess) { rc = fail(QNN_ERR_CUDA, "qnn_mlp_forward_host: stream wait failed"); break; }
            rc = run_mlp(x_dev + r0 * K0, rows, in_bits, layers, L, s_dev + r0 * NL, algo, base, p, st);
        }
        if (rc != QNN_OK) {
            cudaStreamSynchronize(cs);
            cudaStreamSynchronize(st);
        }
        // (events may be destroyed while work that uses them is pending: the runtime frees them when it is done)
        for (int c = 0; c <= chunks; ++c)
            if (ev[c]) cudaEventDestroy(ev[c]);
        if (rc != QNN_OK) return rc;
    }
    QNN_CUDA(cudaMemcpyAsync(scores_host, s_dev, sizeof(int32_t) * (size_t)M * (size_t)NL, cudaMemcpyDeviceToHost, st));
    return QNN_OK;
}

}  // namespace
}  // namespace qnn

using namespace qnn;

extern "C" {

int qnn_mlp_layer_form(const qnn_mlp_layer *layers, int L, int l, int in_bits)
{
    if (layers == nullptr || l < 0 || l >= L || in_bits < 1 || in_bits > 8) return 0;
    return tc_pick_form(l == 0 ? in_bits : 1, l == 0 ? QNN_MODE_U01 : QNN_MODE_PM1, 1, QNN_MODE_PM1, layers[l].K);
}

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

    // Batch rows are independent, so the batch is cut into chunks whose host-to-device copies (on a copy stream
    // of the library's own) run while the previous chunk is being computed on the caller's stream.
    const int chunks = M >= 4096 ? 2 : 1;      // (issued call by call, more chunks cost more in launches than they hide in copies)
    if (int rc = issue_host_pass(x_host, M, in_bits, layers, L, scores_host, algo, base, p, chunks, st)) return rc;
    QNN_CUDA(cudaStreamSynchronize(st));
    return QNN_OK;
}

}  // extern "C"

// A whole pass from host buffers as ONE CUDA graph: built once (stream capture of the same calls
// qnn_mlp_forward_host issues), replayed with a single launch per pass.
struct qnn_mlp_graph {
    cudaGraphExec_t exec;
    int device;
};

extern "C" {

int qnn_mlp_graph_create(const uint8_t *x_host, int64_t M, int in_bits, const qnn_mlp_layer *layers, int L, int32_t *scores_host,
                         int algo, void *ws, size_t ws_bytes, int chunks, void *stream, qnn_mlp_graph **out)
{
    QNN_REQUIRE(out != nullptr, QNN_ERR_INVALID_ARG, "qnn_mlp_graph_create: out is NULL");
    *out = nullptr;
    MlpPlan p;
    if (int rc = plan_mlp(M, in_bits, layers, L, algo, 1, &p)) return rc;
    QNN_REQUIRE(M >= 1, QNN_ERR_INVALID_ARG, "qnn_mlp_graph_create: empty batch");
    QNN_REQUIRE(x_host && scores_host, QNN_ERR_INVALID_ARG, "qnn_mlp_graph_create: NULL input or output");
    QNN_REQUIRE(chunks >= 1 && chunks <= 8, QNN_ERR_INVALID_ARG, "qnn_mlp_graph_create: chunks must be in 1..8");
    QNN_REQUIRE(ws && aligned(ws, 256) && ws_bytes >= p.total, QNN_ERR_WORKSPACE,
                "qnn_mlp_graph_create: workspace of at least %zu bytes (256-byte aligned) required", p.total);
    cudaStream_t st = as_stream(stream);
    QNN_REQUIRE(st != nullptr, QNN_ERR_INVALID_ARG, "qnn_mlp_graph_create: a stream other than the default stream is required for capture");
    char *base = static_cast<char *>(ws);
    // one eager pass first: one-time kernel attributes are set outside the capture, and argument errors surface here
    if (int rc = issue_host_pass(x_host, M, in_bits, layers, L, scores_host, algo, base, p, chunks, st)) return rc;
    QNN_CUDA(cudaStreamSynchronize(st));
    QNN_CUDA(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
    const int rc = issue_host_pass(x_host, M, in_bits, layers, L, scores_host, algo, base, p, chunks, st);
    cudaGraph_t graph = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(st, &graph);
    if (rc != QNN_OK) {
        if (graph) cudaGraphDestroy(graph);
        return rc;
    }
    if (ce != cudaSuccess || graph == nullptr) return fail(QNN_ERR_CUDA, "qnn_mlp_graph_create: stream capture failed: %s", cudaGetErrorString(ce));
    cudaGraphExec_t exec = nullptr;
    const cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ie != cudaSuccess) return fail(QNN_ERR_CUDA, "qnn_mlp_graph_create: cudaGraphInstantiate failed: %s", cudaGetErrorString(ie));
    qnn_mlp_graph *g = new (std::nothrow) qnn_mlp_graph;
    if (g == nullptr) { cudaGraphExecDestroy(exec); return fail(QNN_ERR_CUDA, "qnn_mlp_graph_create: out of host memory"); }
    g->exec = exec;
    g->device = 0;
    cudaGetDevice(&g->device);
    *out = g;
    return QNN_OK;
}

int qnn_mlp_graph_launch(qnn_mlp_graph *g, void *stream)
{
    QNN_REQUIRE(g != nullptr && g->exec != nullptr, QNN_ERR_INVALID_ARG, "qnn_mlp_graph_launch: NULL graph");
    QNN_CUDA(cudaGraphLaunch(g->exec, as_stream(stream)));
    return QNN_OK;
}

int qnn_mlp_graph_destroy(qnn_mlp_graph *g)
{
    if (g == nullptr) return QNN_OK;
    if (g->exec) cudaGraphExecDestroy(g->exec);
    delete g;
    return QNN_OK;
}

}  // extern "C"
