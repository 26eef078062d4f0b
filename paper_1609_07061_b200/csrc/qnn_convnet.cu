// The layer types of the CIFAR-10 ConvNet (Table 7) around the binary convolution, and a runner that chains
// them on one stream: the first convolution on 8-bit pixel codes (Eq. 8 recomposed: codes x +-1 filters on the
// int8 tensor-core path), 2 x 2 max-pooling between a convolution and its folded batch-norm threshold, and the
// fully connected head of Algorithm 4.
#include <cstdlib>
#include "qnn_internal.cuh"

namespace qnn {
namespace {

inline int grid_for(int64_t total)
{
    const int64_t need = ceil_div(total, 256);
    const int64_t cap = (int64_t)sm_count() * 16;
    return (int)(need < cap ? need : cap);
}

// im2col of an NCHW uint8 image: row m = (b, yo, xo) holds the KH*KW*C codes under the filter, k = (kh*KW + kw)*C + c,
// rows P bytes apart (P a multiple of 16), bytes k >= K zero.  A tap outside the image reads pad_code.
// One thread per 16-byte piece of a row.
__global__ void __launch_bounds__(256) im2col_u8_kernel(const uint8_t *__restrict__ x, int C, int H, int W, int KH, int KW,
                                                        int pad, int pad_code, int Ho, int Wo, uint8_t *__restrict__ dst, int P,
                                                        int64_t total)
{
    griddep_launch_dependents();
    griddep_wait();
    const int K = KH * KW * C;
    const int pieces = P >> 4;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int piece = (int)(e % pieces);
        int64_t t = e / pieces;
        const int xo = (int)(t % Wo); t /= Wo;
        const int yo = (int)(t % Ho);
        const int64_t b = t / Ho;
        uint32_t o[4] = {0u, 0u, 0u, 0u};
        // (kh, kw, c) of the first byte by division, of the others by counting on
        int k = piece * 16;
        int tap = k / C, c = k - tap * C;
        int kh = tap / KW, kw = tap - kh * KW;
        const uint8_t *img = x + b * C * H * W;
#pragma unroll
        for (int j = 0; j < 16; ++j, ++k) {
            if (k < K) {
                const int yi = yo + kh - pad, xi = xo + kw - pad;
                uint32_t v = (uint32_t)pad_code;
                if (yi >= 0 && yi < H && xi >= 0 && xi < W) v = __ldg(img + (c * H + yi) * W + xi);
                o[j >> 2] |= v << (8 * (j & 3));
                if (++c == C) {
                    c = 0;
                    if (++kw == KW) { kw = 0; ++kh; }
                }
            }
        }
        reinterpret_cast<uint4 *>(dst)[e] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// Packed filter bank [Cout, taps*Cw] (bit c%32 of word tap*Cw + c/32) -> int8 rows [Cout, P]: +1 -> 0x01, -1 -> 0xFF
// at k = tap*C + c, bytes k >= K zero.  One thread per 16-byte piece.
__global__ void __launch_bounds__(256) conv_u8_weights_kernel(const uint32_t *__restrict__ w, int C, int taps, uint8_t *__restrict__ dst,
                                                              int P, int64_t total)
{
    const int K = taps * C;
    const int Cw = (C + 31) >> 5;
    const int pieces = P >> 4;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int piece = (int)(e % pieces);
        const int64_t co = e / pieces;
        uint32_t o[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const int k = piece * 16 + j;
            if (k < K) {
                const int tap = k / C, c = k - tap * C;
                const uint32_t bit = (__ldg(w + (co * taps + tap) * Cw + (c >> 5)) >> (c & 31)) & 1u;
                o[j >> 2] |= (bit ? 0x01u : 0xFFu) << (8 * (j & 3));
            }
        }
        reinterpret_cast<uint4 *>(dst)[e] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// 2 x 2 / stride 2 max-pooling applied to thresholded bits.  The threshold is monotone in the sum, so the bit of a
// window's largest sum is the OR of the four bits, and the AND for channels whose comparison is flipped.
// One thread per output word (32 channels of one pooled pixel); writes packed bits and / or the same signs as
// tensor-core values (dense NHWC: 32*Cw elements per pixel).
__global__ void __launch_bounds__(256) maxpool2x2_bits_kernel(const uint32_t *__restrict__ in, int H, int W, int Cw, int C,
                                                              const uint8_t *__restrict__ flip, uint32_t *__restrict__ out_bits,
                                                              uint8_t *__restrict__ out_form, int kind, int64_t total)
{
    __shared__ uint32_t fmask[64];
    griddep_launch_dependents();
    for (int cw = threadIdx.x; cw < Cw; cw += blockDim.x) {
        uint32_t m = 0;
        if (flip != nullptr)
            for (int j = 0; j < 32; ++j) {
                const int c = cw * 32 + j;
                if (c < C && __ldg(flip + c) != 0) m |= 1u << j;
            }
        fmask[cw] = m;
    }
    __syncthreads();
    griddep_wait();                                  // the flips above are constants; the bits below are the previous kernel's
    const int Ho = H >> 1, Wo = W >> 1;
    const uint32_t tail = (C & 31) ? ((1u << (C & 31)) - 1u) : 0xffffffffu;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int cw = (int)(e % Cw);
        int64_t t = e / Cw;
        const int xo = (int)(t % Wo); t /= Wo;
        const int yo = (int)(t % Ho);
        const int64_t b = t / Ho;
        const uint32_t *p = in + ((b * H + 2 * yo) * W + 2 * xo) * Cw + cw;
        const uint32_t q0 = __ldg(p), q1 = __ldg(p + Cw), q2 = __ldg(p + (int64_t)W * Cw), q3 = __ldg(p + (int64_t)W * Cw + Cw);
        const uint32_t f = fmask[cw];
        const uint32_t valid = (cw == Cw - 1) ? tail : 0xffffffffu;
        const uint32_t w = (((q0 | q1 | q2 | q3) & ~f) | ((q0 & q1 & q2 & q3) & f)) & valid;
        if (out_bits != nullptr) out_bits[e] = w;
        if (out_form != nullptr) {
            if (kind == QNN_FORM_FP4) {
                reinterpret_cast<uint4 *>(out_form)[e] = signs_to_fp4(w, valid);
            } else {
                uint4 lo, hi;
                signs_to_i8(w, valid, lo, hi);
                reinterpret_cast<uint4 *>(out_form)[2 * e] = lo;
                reinterpret_cast<uint4 *>(out_form)[2 * e + 1] = hi;
            }
        }
    }
}

// ---- first-layer convolution -----------------------------------------------------------------------------------------

struct ConvU8Layout {
    int Ho, Wo;
    int64_t M, K;
    int Pa, Pb;                 // row pitches (bytes) of the im2col matrix and of the int8 filter rows
    size_t col_bytes, w_bytes;
};

bool conv_u8_layout(int B, int C, int H, int W, int Cout, int KH, int KW, int pad, ConvU8Layout *l)
{
    if (B < 0 || C < 1 || H < 1 || W < 1 || Cout < 1 || KH < 1 || KW < 1 || pad < 0) return false;
    if (H + 2 * pad < KH || W + 2 * pad < KW) return false;
    l->Ho = H + 2 * pad - KH + 1;
    l->Wo = W + 2 * pad - KW + 1;
    l->M = (int64_t)B * l->Ho * l->Wo;
    l->K = (int64_t)KH * KW * C;
    if (l->K > 8192) return false;                       // 255 * K stays far below 2^31; rows stay short
    l->Pa = (int)round_up((size_t)l->K, 16);
    l->Pb = (int)tc_row_pitch(ceil_div(l->K, 32), QNN_FORM_I8);
    l->col_bytes = round_up((size_t)l->M * (size_t)l->Pa, 256);
    l->w_bytes = round_up((size_t)Cout * (size_t)l->Pb, 256);
    return true;
}

int conv_u8_prepare_into(const uint32_t *w, int Cout, int C, int KH, int KW, const ConvU8Layout &l, uint8_t *dst, cudaStream_t st)
{
    const int64_t total = (int64_t)Cout * (l.Pb / 16);
    conv_u8_weights_kernel<<<grid_for(total), 256, 0, st>>>(w, C, KH * KW, dst, l.Pb, total);
    return check_launch("first-layer filter rows");
}

struct ConvOut {
    int32_t *out_nchw;
    const int32_t *thr;
    const uint8_t *flip;
    uint32_t *out_bits;
    void *out_form;
    int out_form_kind;
};

// x: uint8 [B,C,H,W]; wf: int8 filter rows (conv_u8_prepare_into); col: im2col scratch of l.col_bytes.
int conv_u8_run(const uint8_t *x, int B, int C, int H, int W, const uint8_t *wf, int Cout, int KH, int KW, int pad, int pad_code,
                const ConvU8Layout &l, const ConvOut &o, uint8_t *col, cudaStream_t st)
{
    if (l.M == 0) return QNN_OK;
    const int64_t total = l.M * (l.Pa / 16);
    QNN_CUDA(launch_pdl(im2col_u8_kernel, dim3(grid_for(total)), dim3(256), 0, st, x, C, H, W, KH, KW, pad, pad_code, l.Ho, l.Wo, col, l.Pa, total));
    if (int rc = check_launch("first-layer im2col")) return rc;
    GemmArgs g{};
    g.ka = 8; g.a_mode = QNN_MODE_U01; g.kb = 1; g.b_mode = QNN_MODE_PM1;
    g.M = l.M; g.N = Cout; g.K = l.K;
    g.a_tc = col; g.a_tc_form = QNN_FORM_I8; g.a_tc_ld = l.Pa;
    g.b_tc = wf; g.b_tc_form = QNN_FORM_I8; g.b_tc_ld = l.Pb;
    g.epilogue = EPI_NCHW; g.out = o.out_nchw; g.hw = (int64_t)l.Ho * l.Wo;
    g.thr = o.thr; g.flip = o.flip; g.out_bits = o.out_bits; g.ld_bits = ceil_div(Cout, 32);
    if (o.out_form) {
        g.out_form = o.out_form; g.out_form_kind = o.out_form_kind;
        g.ld_form = tc_row_bytes(ceil_div(Cout, 32), o.out_form_kind);
    }
    if (int rc = validate_gemm(g)) return rc;
    return launch_gemm_tc(g, QNN_FORM_I8, nullptr, 0, st);
}

int maxpool_run(const uint32_t *bits, int B, int H, int W, int C, const uint8_t *flip, uint32_t *out_bits, void *out_form,
                int out_form_kind, cudaStream_t st)
{
    const int Cw = (int)ceil_div(C, 32);
    const int64_t total = (int64_t)B * (H / 2) * (W / 2) * Cw;
    if (total == 0) return QNN_OK;
    QNN_CUDA(launch_pdl(maxpool2x2_bits_kernel, dim3(grid_for(total)), dim3(256), 0, st, bits, H, W, Cw, C, flip, out_bits,
                        static_cast<uint8_t *>(out_form), out_form_kind, total));
    return check_launch("qnn_maxpool2x2_bits");
}

// ---- the network runner ----------------------------------------------------------------------------------------------

constexpr int MAX_NET_LAYERS = 64;

struct LayerPlan {
    int H, W;                   // conv: input image; FC: 0
    int Ho, Wo;                 // conv: output image after pooling
    bool fast;                  // conv: implicit tensor-core path with a prepared bank
    ConvPrep prep;              // fast conv
    ConvU8Layout u8;            // first-layer conv
    size_t prep_off, prep_bytes;
    int64_t out_rows;           // rows (pixels or batch rows) this layer hands on
    int out_cw;                 // words per row it hands on
    // FC: how its input rows are laid out
    int64_t kwords, pad_period;
    int pad_tail;
    int fc_form;                // FC: tensor-core form its prepared weights are kept in (0 = none)
    int64_t fc_pitch;           // bytes between prepared weight rows
    bool fc_tc;                 // FC: runs on the tensor cores at this batch size
};

struct NetPlan {
    LayerPlan l[MAX_NET_LAYERS];
    size_t prepared_bytes;
    size_t off_col, off_pre, off_act[2], off_gen, gen_bytes, act_bits_bytes, total;
};

int plan_net(int B, int H, int W, const qnn_net_layer *layers, int n, NetPlan *p)
{
    QNN_REQUIRE(layers != nullptr && n >= 1 && n <= MAX_NET_LAYERS, QNN_ERR_INVALID_ARG, "convnet: need 1..%d layers", MAX_NET_LAYERS);
    QNN_REQUIRE(B >= 0 && H >= 1 && W >= 1, QNN_ERR_INVALID_ARG, "convnet: bad batch or image size");
    QNN_REQUIRE(layers[n - 1].kind == QNN_LAYER_FC, QNN_ERR_UNSUPPORTED, "convnet: the last layer must be fully connected");
    int h = H, w = W;
    int64_t feat = 0;             // FC inputs available from the previous layer
    int prev_c = 0;               // channels of the previous conv (0 after an FC layer)
    size_t prep = 0, col = 0, pre = 0, bits = 0, form = 0, gen = 0;
    for (int i = 0; i < n; ++i) {
        const qnn_net_layer &ly = layers[i];
        LayerPlan &lp = p->l[i];
        lp = LayerPlan{};
        QNN_REQUIRE(ly.w != nullptr && ly.C >= 1 && ly.Cout >= 1, QNN_ERR_INVALID_ARG, "convnet: layer %d has bad sizes or NULL weights", i);
        QNN_REQUIRE(i == n - 1 || ly.thr != nullptr, QNN_ERR_INVALID_ARG, "convnet: layer %d needs thresholds", i);
        lp.prep_off = prep;
        if (ly.kind == QNN_LAYER_CONV_U8 || ly.kind == QNN_LAYER_CONV) {
            QNN_REQUIRE(ly.ksize == 2 * ly.pad + 1 && ly.pad >= 0, QNN_ERR_UNSUPPORTED, "convnet: layer %d is not a 'same' convolution", i);
            QNN_REQUIRE(ly.kind == QNN_LAYER_CONV_U8 ? i == 0 : (i > 0 && prev_c == ly.C), QNN_ERR_INVALID_ARG,
                        "convnet: layer %d does not fit its input (channels, or a pixel-code layer that is not first)", i);
            QNN_REQUIRE(!ly.pool || (h >= 2 && w >= 2), QNN_ERR_INVALID_ARG, "convnet: layer %d pools an image smaller than 2 x 2", i);
            lp.H = h; lp.W = w;
            const int64_t M = (int64_t)B * h * w;
            const int cwo = (int)ceil_div(ly.Cout, 32);
            QNN_REQUIRE(cwo <= 64, QNN_ERR_UNSUPPORTED, "convnet: at most 2048 channels");
            if (ly.kind == QNN_LAYER_CONV_U8) {
                QNN_REQUIRE(conv_u8_layout(B, ly.C, h, w, ly.Cout, ly.ksize, ly.ksize, ly.pad, &lp.u8), QNN_ERR_UNSUPPORTED,
                            "convnet: first layer too large (KH*KW*C <= 8192)");
                lp.prep_bytes = lp.u8.w_bytes;
                if (lp.u8.col_bytes > col) col = lp.u8.col_bytes;
            } else {
                lp.fast = conv_prep_layout(ly.Cout, ly.C, ly.ksize, ly.ksize, ly.pad, 0, &lp.prep) && w <= 128;
                if (lp.fast) {
                    lp.prep_bytes = lp.prep.w_bytes + lp.prep.c_bytes;
                } else {
                    const size_t g = qnn_workspace_bytes(QNN_OP_CONV2D, M, ly.Cout, (int64_t)ly.ksize * ly.ksize * 32 * ceil_div(ly.C, 32), 1, 1, QNN_ALGO_AUTO) +
                                     qnn_conv_prepared_bytes(ly.Cout, ly.C, ly.ksize, ly.ksize, ly.pad) + 4096;
                    if (g > gen) gen = g;
                }
            }
            if (ly.pool) {
                const size_t pb = round_up((size_t)M * cwo * 4, 256);
                if (pb > pre) pre = pb;
                h /= 2; w /= 2;
            }
            lp.Ho = h; lp.Wo = w;
            lp.out_rows = (int64_t)B * h * w;
            lp.out_cw = cwo;
            prev_c = ly.Cout;
            feat = (int64_t)h * w * ly.Cout;
        } else if (ly.kind == QNN_LAYER_FC) {
            QNN_REQUIRE(i > 0 && ly.C == feat, QNN_ERR_INVALID_ARG, "convnet: layer %d has %d inputs, the previous layer hands on %lld", i,
                        ly.C, (long long)feat);
            if (prev_c > 0) {
                // rows are feature maps in (h, w, c) order, every pixel padded to whole words
                const int cw = (int)ceil_div(prev_c, 32);
                lp.kwords = (int64_t)h * w * cw;
                lp.pad_period = cw;
                lp.pad_tail = prev_c - 32 * (cw - 1);
            } else {
                lp.kwords = ceil_div(ly.C, 32);
            }
            // weights are also kept in tensor-core form; with both operands ready the tensor cores win from about
            // 2^24 products on (no operand-rewriting launches), below that the CUDA-core kernel's shorter start does
            lp.fc_form = tc_pick_form(1, QNN_MODE_PM1, 1, QNN_MODE_PM1, ly.C);
            if (lp.fc_form != 0) {
                lp.fc_pitch = tc_row_pitch(lp.kwords, lp.fc_form);
                lp.prep_bytes = (size_t)ly.Cout * (size_t)lp.fc_pitch;
                lp.fc_tc = (double)B * (double)ly.Cout * (double)ly.C >= 16777216.0;
            }
            lp.out_rows = B;
            lp.out_cw = (int)ceil_div(ly.Cout, 32);
            prev_c = 0;
            feat = ly.Cout;
        } else {
            return fail(QNN_ERR_INVALID_ARG, "convnet: layer %d has an unknown kind %d", i, ly.kind);
        }
        prep += round_up(lp.prep_bytes, 256);
        if (i < n - 1) {
            const size_t bb = round_up((size_t)lp.out_rows * lp.out_cw * 4, 256);
            const size_t fb = round_up((size_t)lp.out_rows * round_up((size_t)lp.out_cw * 32, 128), 256);   // rows on 128-byte lines
            if (bb > bits) bits = bb;
            if (fb > form) form = fb;
        }
    }
    p->prepared_bytes = prep;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += round_up(bytes > 0 ? bytes : 1, 256); return o; };
    p->off_col = take(col);
    p->off_pre = take(pre);
    p->act_bits_bytes = bits > 0 ? bits : 256;
    p->off_act[0] = take(p->act_bits_bytes + form);
    p->off_act[1] = take(p->act_bits_bytes + form);
    p->gen_bytes = gen;
    p->off_gen = take(gen);
    p->total = off;
    return QNN_OK;
}

}  // namespace
}  // namespace qnn

using namespace qnn;

extern "C" {

size_t qnn_conv2d_u8_workspace_bytes(int B, int C, int H, int W, int Cout, int KH, int KW, int pad)
{
    ConvU8Layout l{};
    if (!conv_u8_layout(B, C, H, W, Cout, KH, KW, pad, &l)) return 0;
    return l.col_bytes + l.w_bytes;
}

int qnn_conv2d_u8(const uint8_t *x, int B, int C, int H, int W, const uint32_t *w, int Cout, int KH, int KW, int pad, int pad_code,
                  int32_t *out_nchw, const int32_t *thr, const uint8_t *flip, uint32_t *out_bits, void *out_form, int out_form_kind,
                  void *ws, size_t ws_bytes, void *stream)
{
    QNN_REQUIRE(B >= 0 && C >= 1 && H >= 1 && W >= 1 && Cout >= 1 && KH >= 1 && KW >= 1 && pad >= 0, QNN_ERR_INVALID_ARG,
                "qnn_conv2d_u8: bad size");
    QNN_REQUIRE(pad_code >= 0 && pad_code <= 255, QNN_ERR_INVALID_ARG, "qnn_conv2d_u8: pad_code must be a uint8 value");
    if (B == 0) return QNN_OK;
    QNN_REQUIRE(x && w, QNN_ERR_INVALID_ARG, "qnn_conv2d_u8: NULL operand");
    QNN_REQUIRE(out_nchw || out_bits || out_form, QNN_ERR_INVALID_ARG, "qnn_conv2d_u8: no output buffer");
    QNN_REQUIRE(!(out_bits || out_form) || thr, QNN_ERR_INVALID_ARG, "qnn_conv2d_u8: thresholds required");
    ConvU8Layout l{};
    QNN_REQUIRE(conv_u8_layout(B, C, H, W, Cout, KH, KW, pad, &l), QNN_ERR_UNSUPPORTED,
                "qnn_conv2d_u8: filter larger than the padded image, or KH*KW*C above 8192");
    QNN_REQUIRE(ws != nullptr && aligned(ws, 256) && ws_bytes >= l.col_bytes + l.w_bytes, QNN_ERR_WORKSPACE,
                "qnn_conv2d_u8: workspace of at least %zu bytes (256-byte aligned) required", l.col_bytes + l.w_bytes);
    cudaStream_t st = as_stream(stream);
    uint8_t *col = static_cast<uint8_t *>(ws);
    uint8_t *wf = col + l.col_bytes;
    if (int rc = conv_u8_prepare_into(w, Cout, C, KH, KW, l, wf, st)) return rc;
    ConvOut o{out_nchw, thr, flip, out_bits, out_form, out_form_kind};
    return conv_u8_run(x, B, C, H, W, wf, Cout, KH, KW, pad, pad_code, l, o, col, st);
}

int qnn_maxpool2x2_bits(const uint32_t *bits, int B, int H, int W, int C, const uint8_t *flip, uint32_t *out_bits, void *out_form,
                        int out_form_kind, void *stream)
{
    QNN_REQUIRE(B >= 0 && H >= 0 && W >= 0 && C >= 1, QNN_ERR_INVALID_ARG, "qnn_maxpool2x2_bits: bad size");
    QNN_REQUIRE(C <= 2048, QNN_ERR_UNSUPPORTED, "qnn_maxpool2x2_bits: at most 2048 channels");
    if (B == 0 || H < 2 || W < 2) return QNN_OK;
    QNN_REQUIRE(bits && (out_bits || out_form), QNN_ERR_INVALID_ARG, "qnn_maxpool2x2_bits: NULL input or no output");
    QNN_REQUIRE(!out_form || out_form_kind == QNN_FORM_I8 || out_form_kind == QNN_FORM_FP4, QNN_ERR_INVALID_ARG,
                "qnn_maxpool2x2_bits: bad output form");
    QNN_REQUIRE(aligned(bits, 4) && aligned(out_bits, 4) && aligned(out_form, 16), QNN_ERR_ALIGNMENT,
                "qnn_maxpool2x2_bits: bits need 4-byte, form output 16-byte alignment");
    return maxpool_run(bits, B, H, W, C, flip, out_bits, out_form, out_form_kind, as_stream(stream));
}

size_t qnn_convnet_prepared_bytes(int H, int W, const qnn_net_layer *layers, int n)
{
    static thread_local NetPlan p;
    if (plan_net(1, H, W, layers, n, &p) != QNN_OK) return 0;
    return p.prepared_bytes > 0 ? p.prepared_bytes : 256;
}

size_t qnn_convnet_workspace_bytes(int B, int H, int W, const qnn_net_layer *layers, int n)
{
    static thread_local NetPlan p;
    if (plan_net(B, H, W, layers, n, &p) != QNN_OK) return 0;
    return p.total;
}

int qnn_convnet_prepare(int H, int W, const qnn_net_layer *layers, int n, void *prepared, size_t prepared_bytes, void *stream)
{
    static thread_local NetPlan p;
    if (int rc = plan_net(1, H, W, layers, n, &p)) return rc;
    QNN_REQUIRE(prepared != nullptr && aligned(prepared, 256) && prepared_bytes >= p.prepared_bytes, QNN_ERR_WORKSPACE,
                "qnn_convnet_prepare: buffer of at least %zu bytes (256-byte aligned) required", p.prepared_bytes);
    cudaStream_t st = as_stream(stream);
    uint8_t *base = static_cast<uint8_t *>(prepared);
    for (int i = 0; i < n; ++i) {
        const qnn_net_layer &ly = layers[i];
        const LayerPlan &lp = p.l[i];
        if (ly.kind == QNN_LAYER_CONV_U8) {
            if (int rc = conv_u8_prepare_into(ly.w, ly.Cout, ly.C, ly.ksize, ly.ksize, lp.u8, base + lp.prep_off, st)) return rc;
        } else if (ly.kind == QNN_LAYER_CONV && lp.fast) {
            if (int rc = qnn_conv_prepare(ly.w, ly.Cout, ly.C, ly.ksize, ly.ksize, ly.pad, 1, base + lp.prep_off, lp.prep_bytes, stream))
                return rc;
        } else if (ly.kind == QNN_LAYER_FC && lp.fc_form != 0) {
            const int64_t period = lp.pad_period > 0 ? lp.pad_period : lp.kwords;
            const int tail = lp.pad_period > 0 ? lp.pad_tail : (int)(ly.C - 32 * (lp.kwords - 1));
            if (int rc = tc_expand(ly.w, 1, QNN_MODE_PM1, lp.kwords, 0, ly.Cout, lp.kwords, period, tail, lp.fc_form, base + lp.prep_off,
                                   lp.fc_pitch, st))
                return rc;
        }
    }
    return QNN_OK;
}

int qnn_convnet_forward(const uint8_t *x, int B, int H, int W, const qnn_net_layer *layers, int n, const void *prepared,
                        int32_t *scores, void *ws, size_t ws_bytes, void *stream)
{
    static thread_local NetPlan p;
    if (int rc = plan_net(B, H, W, layers, n, &p)) return rc;
    if (B == 0) return QNN_OK;
    QNN_REQUIRE(x && scores && prepared, QNN_ERR_INVALID_ARG, "qnn_convnet_forward: NULL input, output or prepared weights");
    QNN_REQUIRE(aligned(prepared, 256), QNN_ERR_ALIGNMENT, "qnn_convnet_forward: prepared weights must be 256-byte aligned");
    QNN_REQUIRE(ws && aligned(ws, 256) && ws_bytes >= p.total, QNN_ERR_WORKSPACE,
                "qnn_convnet_forward: workspace of at least %zu bytes (256-byte aligned) required", p.total);
    cudaStream_t st = as_stream(stream);
    char *wsb = static_cast<char *>(ws);
    const uint8_t *prep = static_cast<const uint8_t *>(prepared);
    uint32_t *pre = reinterpret_cast<uint32_t *>(wsb + p.off_pre);
    void *gen = wsb + p.off_gen;

    // what the previous layer left for this one
    const uint32_t *cur_bits = nullptr;
    const void *cur_form = nullptr;
    int cur_kind = 0;
    int64_t cur_form_ld = 0;
    // the form layer i reads its input in: a tensor-core layer its operand form, everything else packed bits (0)
    auto in_form = [&](int i) -> int {
        if (i >= n) return 0;
        if (layers[i].kind == QNN_LAYER_CONV && p.l[i].fast) return p.l[i].prep.form;
        if (layers[i].kind == QNN_LAYER_FC && p.l[i].fc_tc) return p.l[i].fc_form;
        return 0;
    };

    for (int i = 0; i < n; ++i) {
        const qnn_net_layer &ly = layers[i];
        const LayerPlan &lp = p.l[i];
        const bool last = i == n - 1;
        // what the next layer reads: a fast convolution its form, everything else packed bits
        const int want_form = in_form(i + 1);
        uint32_t *act_bits = reinterpret_cast<uint32_t *>(wsb + p.off_act[i & 1]);
        void *act_form = wsb + p.off_act[i & 1] + p.act_bits_bytes;

        if (ly.kind == QNN_LAYER_FC) {
            GemmArgs g{};
            g.ka = g.kb = 1; g.a_mode = g.b_mode = QNN_MODE_PM1;
            g.M = B; g.N = ly.Cout; g.K = ly.C;
            if (lp.pad_period > 0) { g.kwords = lp.kwords; g.pad_period = lp.pad_period; g.pad_tail = lp.pad_tail; }
            if (last) {
                g.epilogue = EPI_ROWMAJOR; g.out = scores; g.ldo = ly.Cout;
            } else {
                g.epilogue = EPI_BITS; g.thr = ly.thr; g.flip = ly.flip;
                if (want_form != 0 && lp.fc_tc) {
                    g.out_form = act_form; g.out_form_kind = want_form; g.ld_form = tc_row_pitch(lp.out_cw, want_form);
                } else {
                    g.out_bits = act_bits; g.ld_bits = lp.out_cw;
                }
            }
            if (lp.fc_tc && cur_form != nullptr && cur_kind == lp.fc_form) {
                g.a_tc = cur_form; g.a_tc_form = cur_kind; g.a_tc_ld = cur_form_ld;
                g.b_tc = prep + lp.prep_off; g.b_tc_form = lp.fc_form; g.b_tc_ld = lp.fc_pitch;
                if (int rc = validate_gemm(g)) return rc;
                if (int rc = launch_gemm_tc(g, lp.fc_form, nullptr, 0, st)) return rc;
            } else {
                QNN_REQUIRE(cur_bits != nullptr, QNN_ERR_INVALID_ARG, "convnet: layer %d has no packed input", i);
                g.a = cur_bits; g.lda = lp.kwords; g.b = ly.w; g.ldb = lp.kwords;
                if (int rc = run_gemm(g, QNN_ALGO_POPC, nullptr, 0, st)) return rc;
            }
            if (g.out_form != nullptr) {
                cur_bits = nullptr; cur_form = act_form; cur_kind = want_form; cur_form_ld = g.ld_form;
            } else {
                // a CUDA-core layer feeding a tensor-core one: rewrite its bits in the form the next layer reads
                cur_bits = act_bits; cur_form = nullptr; cur_kind = 0;
                if (!last && want_form != 0) {
                    const int64_t cw = lp.out_cw, ld = tc_row_pitch(cw, want_form);
                    if (int rc = tc_expand(act_bits, 1, QNN_MODE_PM1, cw, 0, B, cw, cw, ly.Cout - 32 * ((int)cw - 1), want_form,
                                           static_cast<uint8_t *>(act_form), ld, st))
                        return rc;
                    cur_bits = nullptr; cur_form = act_form; cur_kind = want_form; cur_form_ld = ld;
                }
            }
            continue;
        }

        // a convolution: threshold straight to what the next layer reads, or to bits that the pooling step turns into it
        ConvOut o{};
        o.thr = ly.thr; o.flip = ly.flip;
        // narrow images pool inside the convolution's own epilogue; wider ones through packed bits and the pooling kernel
        // (QNN_FUSED_POOL=0 in the environment keeps the pooling kernel everywhere)
        static const bool fuse_ok = [] { const char *e = getenv("QNN_FUSED_POOL"); return !(e && e[0] == '0'); }();
        const bool fused_pool = fuse_ok && ly.pool && ly.kind == QNN_LAYER_CONV && lp.fast && qnn_conv_can_pool(lp.H, lp.W);
        const bool separate_pool = ly.pool && !fused_pool;
        const bool direct_form = want_form != 0 && !separate_pool;
        if (separate_pool) o.out_bits = pre;
        else if (direct_form) { o.out_form = act_form; o.out_form_kind = want_form; }
        else o.out_bits = act_bits;

        if (ly.kind == QNN_LAYER_CONV_U8) {
            if (int rc = conv_u8_run(x, B, ly.C, lp.H, lp.W, prep + lp.prep_off, ly.Cout, ly.ksize, ly.ksize, ly.pad, 0, lp.u8, o,
                                     reinterpret_cast<uint8_t *>(wsb + p.off_col), st))
                return rc;
        } else if (lp.fast) {
            qnn_conv_io io{};
            io.x = cur_form && cur_kind == lp.prep.form ? cur_form : static_cast<const void *>(cur_bits);
            io.x_form = cur_form && cur_kind == lp.prep.form ? cur_kind : 0;
            io.thr = o.thr; io.flip = o.flip; io.out_bits = o.out_bits; io.out_form = o.out_form; io.out_form_kind = o.out_form_kind;
            io.pool2x2 = fused_pool ? 1 : 0;
            QNN_REQUIRE(io.x != nullptr, QNN_ERR_INVALID_ARG, "convnet: layer %d has no input", i);
            if (int rc = qnn_binary_conv2d_prepared(&io, B, ly.C, lp.H, lp.W, prep + lp.prep_off, ly.Cout, ly.ksize, ly.ksize, ly.pad, gen,
                                                    p.gen_bytes, stream))
                return rc;
        } else {
            // any other geometry: packed im2col and the matrix product the library picks; it writes bits only
            uint32_t *dst = separate_pool ? pre : act_bits;
            if (int rc = qnn_binary_conv2d(cur_bits, B, ly.C, lp.H, lp.W, ly.w, ly.Cout, ly.ksize, ly.ksize, 1, ly.pad, 1, nullptr, ly.thr,
                                           ly.flip, dst, QNN_ALGO_AUTO, gen, p.gen_bytes, stream))
                return rc;
            if (direct_form) {
                const int64_t cw = lp.out_cw;
                if (int rc = tc_expand(act_bits, 1, QNN_MODE_PM1, cw, 0, lp.out_rows, cw, cw, ly.Cout - 32 * ((int)cw - 1), want_form,
                                       static_cast<uint8_t *>(act_form), tc_row_bytes(cw, want_form), st))
                    return rc;
            }
        }
        if (separate_pool) {
            if (int rc = maxpool_run(pre, B, lp.H, lp.W, ly.Cout, ly.flip, want_form ? nullptr : act_bits, want_form ? act_form : nullptr,
                                     want_form, st))
                return rc;
        }
        cur_bits = want_form ? nullptr : act_bits;
        cur_form = want_form ? act_form : nullptr;
        cur_kind = want_form;
        cur_form_ld = want_form ? tc_row_bytes(lp.out_cw, want_form) * (layers[i + 1].kind == QNN_LAYER_FC ? (int64_t)lp.Ho * lp.Wo : 1) : 0;
    }
    return QNN_OK;
}

}  // extern "C"
