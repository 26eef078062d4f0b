// Binary convolution (Sec. 5) as a packed im2col followed by the XNOR matrix
// product, plus the weight re-layout and the fp32 affine rescale.
#include "qnn_internal.cuh"

namespace qnn {
namespace {

// One thread per word of the im2col matrix col[m, (kh*KW + kw)*Cw + cw],
// m = (b, yo, xo).  A tap outside the image reads the pad word: all valid
// channel bits set for +1 padding, zero for -1 padding; bits of channels
// >= C stay zero in every word so they cancel against the weights' zero pads.
__global__ void __launch_bounds__(256) im2col_bits_kernel(const uint32_t *__restrict__ x, int B, int C, int H, int W,
                                                          int KH, int KW, int stride, int pad, int pad_bit, int Ho,
                                                          int Wo, uint32_t *__restrict__ col, int64_t total)
{
    const int Cw = (C + 31) >> 5;
    const uint32_t tail_mask = (C & 31) ? ((1u << (C & 31)) - 1u) : 0xffffffffu;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int cw = (int)(e % Cw);
        int64_t t = e / Cw;
        const int kw = (int)(t % KW); t /= KW;
        const int kh = (int)(t % KH); t /= KH;
        const int xo = (int)(t % Wo); t /= Wo;
        const int yo = (int)(t % Ho); t /= Ho;
        const int b = (int)t;
        const int yi = yo * stride + kh - pad;
        const int xi = xo * stride + kw - pad;
        uint32_t v;
        if (yi >= 0 && yi < H && xi >= 0 && xi < W)
            v = __ldg(x + (((int64_t)b * H + yi) * W + xi) * Cw + cw);
        else
            v = pad_bit ? ((cw == Cw - 1) ? tail_mask : 0xffffffffu) : 0u;
        col[e] = v;
    }
}

// One thread per output word out[co, (kh*KW + kw)*Cw + cw]: gathers 32 channels of one filter tap.
__global__ void __launch_bounds__(256) conv_weight_pack_kernel(const float *__restrict__ w, int Cout, int C, int KH,
                                                               int KW, uint32_t *__restrict__ out, int64_t total)
{
    const int Cw = (C + 31) >> 5;
    const int taps = KH * KW;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int cw = (int)(e % Cw);
        int64_t t = e / Cw;
        const int tap = (int)(t % taps);
        const int co = (int)(t / taps);
        uint32_t word = 0;
        for (int j = 0; j < 32; ++j) {
            const int c = cw * 32 + j;
            if (c < C) word |= (uint32_t)(__ldg(w + ((int64_t)co * C + c) * taps + tap) >= 0.0f) << j;
        }
        out[e] = word;
    }
}

// First fully-connected layer after a convolution: w is [H*W*C, N] row-major with its inputs in (h, w, c) order.
// One thread per output word out[n, pix*Cw + cw]; consecutive threads take consecutive n (coalesced reads).
__global__ void __launch_bounds__(256) fc_after_conv_pack_kernel(const float *__restrict__ w, int N, int C, int HW,
                                                                 uint32_t *__restrict__ out, int64_t total)
{
    const int Cw = (C + 31) >> 5;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(e % N);
        const int64_t t = e / N;
        const int cw = (int)(t % Cw);
        const int pix = (int)(t / Cw);
        uint32_t word = 0;
        for (int j = 0; j < 32; ++j) {
            const int c = cw * 32 + j;
            if (c < C) word |= (uint32_t)(__ldg(w + ((int64_t)pix * C + c) * N + n) >= 0.0f) << j;
        }
        out[(int64_t)n * HW * Cw + (int64_t)pix * Cw + cw] = word;
    }
}

__global__ void __launch_bounds__(256) rescale_kernel(const int32_t *__restrict__ p, int64_t M, int64_t N, int64_t ldp,
                                                      float alpha, const float *__restrict__ row_off,
                                                      const float *__restrict__ col_off, float delta,
                                                      float *__restrict__ y, int64_t ldy)
{
    const int64_t total = M * N;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t m = e / N, n = e - m * N;
        float v = __fmul_rn(alpha, (float)p[m * ldp + n]);
        if (row_off) v = __fadd_rn(v, row_off[m]);
        if (col_off) v = __fadd_rn(v, col_off[n]);
        v = __fadd_rn(v, delta);
        y[m * ldy + n] = v;
    }
}

// Border corrections of the implicit-GEMM convolution.  The tensor-core kernel reads out-of-image
// taps as 0; the padding value (+1 or -1) times the weights of those taps is added back here.
// A pixel's class says how many filter rows fall off the top / bottom and how many filter columns
// fall off the left / right: cls = ((ty*(pad+1) + by)*(pad+1) + tx)*(pad+1) + bx.
// corr[cls, co] = (+-1) * sum over out-of-image taps of sum_c w[co, c, tap]; rows are ld = Cout rounded up to 32
// long, the pad columns zero.
__global__ void __launch_bounds__(128) conv_border_corr_kernel(const uint32_t *__restrict__ w, int Cout, int C, int KH, int KW,
                                                               int pad, int pad_bit, int32_t *__restrict__ corr, int classes, int ld)
{
    // one block per output channel (and per pad column): first the sum of every tap's weights, then the classes
    __shared__ int32_t tap_sum[64];
    const int co = blockIdx.x;
    const int taps = KH * KW;
    if (co >= Cout) {
        for (int cls = threadIdx.x; cls < classes; cls += blockDim.x) corr[cls * ld + co] = 0;
        return;
    }
    const int Cw = (C + 31) >> 5;
    for (int t = threadIdx.x; t < taps; t += blockDim.x) tap_sum[t] = 0;
    __syncthreads();
    const uint32_t *wp = w + (int64_t)co * taps * Cw;
    for (int e = threadIdx.x; e < taps * Cw; e += blockDim.x) atomicAdd(&tap_sum[e / Cw], 2 * __popc(__ldg(wp + e)));
    __syncthreads();
    const int pc = pad + 1;
    for (int c0 = threadIdx.x; c0 < classes; c0 += blockDim.x) {
        int cls = c0;
        const int bx = cls % pc; cls /= pc;
        const int tx = cls % pc; cls /= pc;
        const int by = cls % pc; cls /= pc;
        const int ty = cls;
        int32_t sum = 0;
        for (int kh = 0; kh < KH; ++kh)
            for (int kw = 0; kw < KW; ++kw)
                if (kh < ty || kh >= KH - by || kw < tx || kw >= KW - bx) sum += tap_sum[kh * KW + kw] - C;
        corr[c0 * ld + co] = pad_bit ? sum : -sum;
    }
}

inline int grid_for(int64_t total)
{
    const int64_t need = ceil_div(total, 256);
    const int64_t cap = (int64_t)sm_count() * 16;
    return (int)(need < cap ? need : cap);
}

int conv_prepare_into(const uint32_t *w, int Cout, int C, int KH, int KW, int pad, int pad_bit, const ConvPrep &l, uint8_t *wf,
                      int32_t *corr, cudaStream_t st)
{
    if (int rc = tc_expand(w, 1, QNN_MODE_PM1, l.kwords, 0, Cout, l.kwords, l.kwords, 32, l.form, wf, l.w_pitch, st)) return rc;
    conv_border_corr_kernel<<<l.corr_ld, 128, 0, st>>>(w, Cout, C, KH, KW, pad, pad_bit, corr, l.classes, l.corr_ld);
    return check_launch("conv border table");
}

}  // namespace

// The implicit tensor-core path takes stride-1 "same" filters (at most 7 x 7: 64 taps), images at most 128 pixels wide
// and whole channel blocks per pixel: multiples of 128 channels as e2m1 values (128-byte blocks when C is a multiple
// of 256, else 64-byte blocks), or as int8 (128-byte blocks) when that form is asked for.  want_form = 0: the best form.
bool conv_prep_layout(int Cout, int C, int KH, int KW, int pad, int want_form, ConvPrep *l)
{
    if (KH != 2 * pad + 1 || KW != 2 * pad + 1 || pad > 3 || (int64_t)KH * KW * C >= (1 << 24)) return false;
    if (C % 128 != 0) return false;
    const int form = want_form == QNN_FORM_I8 ? QNN_FORM_I8 : QNN_FORM_FP4;
    l->form = form;
    l->kblk = (form == QNN_FORM_FP4 && C % 256 != 0) ? 64 : 128;
    l->kwords = (int64_t)KH * KW * ceil_div(C, 32);
    l->w_pitch = tc_row_pitch(l->kwords, form);
    l->classes = (pad + 1) * (pad + 1) * (pad + 1) * (pad + 1);
    l->corr_ld = (int)round_up((size_t)Cout, 32);
    l->w_bytes = round_up((size_t)Cout * (size_t)l->w_pitch, 256);
    l->c_bytes = round_up(sizeof(int32_t) * (size_t)l->classes * (size_t)l->corr_ld, 256);
    return true;
}

}  // namespace qnn

using namespace qnn;

extern "C" {

int qnn_pack_conv_weights(const float *w, int Cout, int C, int KH, int KW, uint32_t *out, void *stream)
{
    QNN_REQUIRE(Cout >= 0 && C >= 0 && KH >= 1 && KW >= 1, QNN_ERR_INVALID_ARG, "qnn_pack_conv_weights: bad sizes");
    if (Cout == 0 || C == 0) return QNN_OK;
    QNN_REQUIRE(w && out, QNN_ERR_INVALID_ARG, "qnn_pack_conv_weights: NULL pointer");
    const int64_t total = (int64_t)Cout * KH * KW * ceil_div(C, 32);
    conv_weight_pack_kernel<<<grid_for(total), 256, 0, as_stream(stream)>>>(w, Cout, C, KH, KW, out, total);
    return check_launch("qnn_pack_conv_weights");
}

int qnn_pack_fc_after_conv_weights(const float *w, int N, int C, int H, int W, uint32_t *out, void *stream)
{
    QNN_REQUIRE(N >= 0 && C >= 0 && H >= 1 && W >= 1, QNN_ERR_INVALID_ARG, "qnn_pack_fc_after_conv_weights: bad sizes");
    if (N == 0 || C == 0) return QNN_OK;
    QNN_REQUIRE(w && out, QNN_ERR_INVALID_ARG, "qnn_pack_fc_after_conv_weights: NULL pointer");
    const int64_t total = (int64_t)N * H * W * ceil_div(C, 32);
    fc_after_conv_pack_kernel<<<grid_for(total), 256, 0, as_stream(stream)>>>(w, N, C, H * W, out, total);
    return check_launch("qnn_pack_fc_after_conv_weights");
}

int qnn_rescale_f32(const int32_t *p, int64_t M, int64_t N, int64_t ldp, float alpha, const float *row_off,
                    const float *col_off, float delta, float *y, int64_t ldy, void *stream)
{
    QNN_REQUIRE(M >= 0 && N >= 0, QNN_ERR_INVALID_ARG, "qnn_rescale_f32: negative size");
    if (M == 0 || N == 0) return QNN_OK;
    QNN_REQUIRE(p && y, QNN_ERR_INVALID_ARG, "qnn_rescale_f32: NULL pointer");
    QNN_REQUIRE(ldp >= N && ldy >= N, QNN_ERR_INVALID_ARG, "qnn_rescale_f32: leading dimension too small");
    rescale_kernel<<<grid_for(M * N), 256, 0, as_stream(stream)>>>(p, M, N, ldp, alpha, row_off, col_off, delta, y, ldy);
    return check_launch("qnn_rescale_f32");
}

int qnn_binary_conv2d(const uint32_t *x, int B, int C, int H, int W, const uint32_t *w, int Cout, int KH, int KW,
                      int stride, int pad, int pad_bit, int32_t *out_nchw, const int32_t *thr, const uint8_t *flip,
                      uint32_t *out_bits, int algo, void *ws, size_t ws_bytes, void *stream)
{
    QNN_REQUIRE(B >= 0 && C >= 0 && H >= 0 && W >= 0 && Cout >= 0, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d: negative size");
    QNN_REQUIRE(KH >= 1 && KW >= 1 && stride >= 1 && pad >= 0 && (pad_bit == 0 || pad_bit == 1), QNN_ERR_INVALID_ARG,
                "qnn_binary_conv2d: bad kernel, stride, pad or pad_bit");
    if (B == 0 || C == 0 || Cout == 0 || H == 0 || W == 0) return QNN_OK;
    QNN_REQUIRE(H + 2 * pad >= KH && W + 2 * pad >= KW, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d: kernel larger than padded image");
    QNN_REQUIRE(x && w, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d: NULL operand");
    QNN_REQUIRE(out_nchw || out_bits, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d: no output buffer");
    QNN_REQUIRE(!out_bits || thr, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d: thresholds required for packed-bit output");
    const int Ho = (H + 2 * pad - KH) / stride + 1;
    const int Wo = (W + 2 * pad - KW) / stride + 1;
    const int64_t Cw = ceil_div(C, 32);
    const int64_t M = (int64_t)B * Ho * Wo;
    const int64_t kwords = (int64_t)KH * KW * Cw;
    cudaStream_t st = as_stream(stream);
    QNN_REQUIRE(algo >= QNN_ALGO_AUTO && algo <= QNN_ALGO_TC_PACKED, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d: unknown algo %d", algo);

    GemmArgs g{};
    g.b = w; g.ldb = kwords; g.ka = g.kb = 1; g.a_mode = g.b_mode = QNN_MODE_PM1;
    g.M = M; g.N = Cout; g.K = (int64_t)KH * KW * C; g.kwords = kwords;
    g.pad_period = Cw; g.pad_tail = (int)(C - 32 * (Cw - 1));
    g.epilogue = EPI_NCHW; g.out = out_nchw; g.hw = (int64_t)Ho * Wo;
    g.thr = thr; g.flip = flip; g.out_bits = out_bits; g.ld_bits = ceil_div(Cout, 32);

    // ---- implicit GEMM on the tensor cores: no im2col matrix ------------------------------------
    ConvPrep lay{};
    bool implicit = stride == 1 && W <= 128 && algo != QNN_ALGO_POPC && algo != QNN_ALGO_B1_MMA && algo != QNN_ALGO_TC_PACKED &&
                    conv_prep_layout(Cout, C, KH, KW, pad, algo == QNN_ALGO_TC_I8 ? QNN_FORM_I8 : (algo == QNN_ALGO_TC_FP4 ? QNN_FORM_FP4 : 0), &lay);
    if (implicit && algo == QNN_ALGO_AUTO) {
        const int pick = qnn_select_algo(M, Cout, g.K, 1, 1, QNN_MODE_PM1, QNN_MODE_PM1);
        implicit = pick == QNN_ALGO_TC_FP4 || pick == QNN_ALGO_TC_I8 || pick == QNN_ALGO_TC_PACKED;
    }
    if (implicit) {
        const int64_t cbytes = tc_row_bytes(Cw, lay.form);
        const size_t x_bytes = round_up((size_t)M * (size_t)cbytes, 256);
        if (ws != nullptr && aligned(ws, 256) && ws_bytes >= x_bytes + lay.w_bytes + lay.c_bytes) {
            uint8_t *xf = static_cast<uint8_t *>(ws);
            uint8_t *wf = xf + x_bytes;
            int32_t *corr = reinterpret_cast<int32_t *>(wf + lay.w_bytes);
            g.a_tc = xf; g.a_tc_form = lay.form; g.a_tc_ld = cbytes;
            g.b_tc = wf; g.b_tc_form = lay.form; g.b_tc_ld = lay.w_pitch;
            if (int rc = validate_gemm(g)) return rc;
            if (int rc = tc_expand(x, 1, QNN_MODE_PM1, Cw, 0, M, Cw, Cw, 32, lay.form, xf, cbytes, st)) return rc;
            if (int rc = conv_prepare_into(w, Cout, C, KH, KW, pad, pad_bit, lay, wf, corr, st)) return rc;
            ConvImplicit ci{};
            ci.B = B; ci.H = H; ci.W = W; ci.KH = KH; ci.KW = KW; ci.pad = pad;
            ci.cblocks = (int32_t)(cbytes / lay.kblk); ci.kblk = lay.kblk;
            ci.corr = corr;
            g.conv = &ci;
            return launch_gemm_tc(g, lay.form, nullptr, 0, st);
        }
        QNN_REQUIRE(algo == QNN_ALGO_AUTO, QNN_ERR_WORKSPACE,
                    "qnn_binary_conv2d: workspace of at least %zu bytes (256-byte aligned) required", x_bytes + lay.w_bytes + lay.c_bytes);
    }

    // ---- packed im2col + matrix product ------------------------------------------------------------
    const size_t col_bytes = round_up(sizeof(uint32_t) * (size_t)M * (size_t)kwords, 256);
    QNN_REQUIRE(ws != nullptr && aligned(ws, 256) && ws_bytes >= col_bytes, QNN_ERR_WORKSPACE,
                "qnn_binary_conv2d: workspace of at least %zu bytes (256-byte aligned) required", col_bytes);
    uint32_t *col = static_cast<uint32_t *>(ws);
    g.a = col; g.lda = kwords;
    if (int rc = validate_gemm(g)) return rc;

    const int64_t total = M * kwords;
    im2col_bits_kernel<<<grid_for(total), 256, 0, st>>>(x, B, C, H, W, KH, KW, stride, pad, pad_bit, Ho, Wo, col, total);
    if (int rc = check_launch("qnn_binary_conv2d im2col")) return rc;
    return run_gemm(g, algo, static_cast<char *>(ws) + col_bytes, ws_bytes - col_bytes, st);
}

size_t qnn_conv_prepared_bytes(int Cout, int C, int KH, int KW, int pad)
{
    ConvPrep l{};
    if (Cout <= 0 || C <= 0 || !conv_prep_layout(Cout, C, KH, KW, pad, 0, &l)) return 0;
    return l.w_bytes + l.c_bytes;
}

int qnn_conv_prepare(const uint32_t *w, int Cout, int C, int KH, int KW, int pad, int pad_bit, void *prepared, size_t prepared_bytes,
                     void *stream)
{
    QNN_REQUIRE(w && prepared, QNN_ERR_INVALID_ARG, "qnn_conv_prepare: NULL pointer");
    QNN_REQUIRE(Cout >= 1 && C >= 1 && (pad_bit == 0 || pad_bit == 1), QNN_ERR_INVALID_ARG, "qnn_conv_prepare: bad sizes or pad_bit");
    ConvPrep l{};
    QNN_REQUIRE(conv_prep_layout(Cout, C, KH, KW, pad, 0, &l), QNN_ERR_UNSUPPORTED,
                "qnn_conv_prepare: needs a stride-1 'same' filter up to 7 x 7 and C a multiple of 128; use qnn_binary_conv2d");
    QNN_REQUIRE(aligned(prepared, 256) && prepared_bytes >= l.w_bytes + l.c_bytes, QNN_ERR_WORKSPACE,
                "qnn_conv_prepare: buffer of at least %zu bytes (256-byte aligned) required", l.w_bytes + l.c_bytes);
    uint8_t *wf = static_cast<uint8_t *>(prepared);
    return conv_prepare_into(w, Cout, C, KH, KW, pad, pad_bit, l, wf, reinterpret_cast<int32_t *>(wf + l.w_bytes), as_stream(stream));
}

int qnn_conv_can_pool(int H, int W)
{
    return (W == 2 || W == 4 || W == 8 || W == 16) && H >= 2 && H % 2 == 0;
}

int qnn_conv_form(int C)
{
    return C > 0 && C % 128 == 0 ? QNN_FORM_FP4 : 0;
}

int qnn_binary_conv2d_prepared(const qnn_conv_io *io, int B, int C, int H, int W, const void *prepared, int Cout, int KH, int KW,
                               int pad, void *ws, size_t ws_bytes, void *stream)
{
    QNN_REQUIRE(io != nullptr && prepared != nullptr, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d_prepared: NULL descriptor");
    QNN_REQUIRE(B >= 0 && C >= 1 && H >= 0 && W >= 0 && Cout >= 1, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d_prepared: bad size");
    if (B == 0 || H == 0 || W == 0) return QNN_OK;
    ConvPrep l{};
    QNN_REQUIRE(conv_prep_layout(Cout, C, KH, KW, pad, 0, &l) && W <= 128, QNN_ERR_UNSUPPORTED,
                "qnn_binary_conv2d_prepared: needs a stride-1 'same' filter up to 7 x 7, C a multiple of 128 and W <= 128");
    QNN_REQUIRE(io->x != nullptr, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d_prepared: NULL input");
    QNN_REQUIRE(io->x_form == 0 || io->x_form == l.form, QNN_ERR_INVALID_ARG,
                "qnn_binary_conv2d_prepared: input form %d, but this filter bank multiplies in form %d", io->x_form, l.form);
    QNN_REQUIRE(io->out_nchw || io->out_bits || io->out_form, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d_prepared: no output buffer");
    QNN_REQUIRE(!(io->out_bits || io->out_form) || io->thr, QNN_ERR_INVALID_ARG, "qnn_binary_conv2d_prepared: thresholds required");
    QNN_REQUIRE(!io->pool2x2 || (qnn_conv_can_pool(H, W) && io->out_nchw == nullptr), QNN_ERR_UNSUPPORTED,
                "qnn_binary_conv2d_prepared: pooling in the same call needs W in {2,4,8,16}, an even H and no int32 output; "
                "use qnn_maxpool2x2_bits");
    cudaStream_t st = as_stream(stream);
    const int64_t Cw = ceil_div(C, 32);
    const int64_t M = (int64_t)B * H * W;
    const int64_t cbytes = tc_row_bytes(Cw, l.form);
    const uint8_t *wf = static_cast<const uint8_t *>(prepared);

    GemmArgs g{};
    g.ka = g.kb = 1; g.a_mode = g.b_mode = QNN_MODE_PM1;
    g.M = M; g.N = Cout; g.K = (int64_t)KH * KW * C; g.kwords = l.kwords;
    g.pad_period = Cw; g.pad_tail = 32;
    g.epilogue = EPI_NCHW; g.out = io->out_nchw; g.hw = (int64_t)H * W;
    g.thr = io->thr; g.flip = io->flip; g.out_bits = io->out_bits; g.ld_bits = ceil_div(Cout, 32);
    if (io->out_form) {
        g.out_form = io->out_form; g.out_form_kind = io->out_form_kind;
        g.ld_form = tc_row_bytes(ceil_div(Cout, 32), io->out_form_kind);      // dense NHWC: the next layer's pixels
    }
    g.b_tc = wf; g.b_tc_form = l.form; g.b_tc_ld = l.w_pitch;
    if (io->x_form != 0) {
        g.a_tc = io->x;
    } else {
        const size_t x_bytes = round_up((size_t)M * (size_t)cbytes, 256);
        QNN_REQUIRE(ws != nullptr && aligned(ws, 256) && ws_bytes >= x_bytes, QNN_ERR_WORKSPACE,
                    "qnn_binary_conv2d_prepared: workspace of at least %zu bytes (256-byte aligned) required", x_bytes);
        g.a_tc = ws;
    }
    g.a_tc_form = l.form; g.a_tc_ld = cbytes;
    if (int rc = validate_gemm(g)) return rc;
    if (io->x_form == 0)
        if (int rc = tc_expand(static_cast<const uint32_t *>(io->x), 1, QNN_MODE_PM1, Cw, 0, M, Cw, Cw, 32, l.form,
                               static_cast<uint8_t *>(ws), cbytes, st))
            return rc;
    ConvImplicit ci{};
    ci.B = B; ci.H = H; ci.W = W; ci.KH = KH; ci.KW = KW; ci.pad = pad;
    ci.cblocks = (int32_t)(cbytes / l.kblk); ci.kblk = l.kblk;
    ci.pool = io->pool2x2 ? 1 : 0;
    ci.corr = reinterpret_cast<const int32_t *>(wf + l.w_bytes);
    g.conv = &ci;
    return launch_gemm_tc(g, l.form, nullptr, 0, st);
}

}  // extern "C"
