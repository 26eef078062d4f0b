/*
 * qnn.h -- C ABI of the B200 (sm_100a) quantised-network forward library.
 *
 * The library implements the inference hot path of quantised / binarised
 * neural networks: sign and k-bit linear quantisation of real tensors,
 * bit-packing along the reduction dimension K, the 1-bit x 1-bit
 * XNOR-popcount matrix product, k-bit operands as weighted sums of bit-plane
 * products, batch-norm + sign folded to a per-channel integer threshold that
 * emits packed bits for the next layer, and binary convolution through a
 * packed im2col matrix.
 *
 * Conventions (all entry points):
 *  - Every function returns an int status (QNN_OK = 0 or a QNN_ERR_* code),
 *    never throws, aborts or traps.  qnn_last_error() returns a thread-local
 *    text for the last failure.  Arguments (pointers, sizes, alignment,
 *    workspace) are validated on the host BEFORE anything is launched: a call
 *    that returns an argument error launched nothing.  QNN_ERR_CUDA is the one
 *    exception: a runtime or driver call that fails part-way through a call
 *    made of several kernels may leave the earlier ones queued.
 *    When QNN_ALGO_AUTO has to leave its preferred algorithm (no workspace, a
 *    misaligned one), the call still returns QNN_OK and qnn_last_error() holds
 *    a note saying which algorithm ran instead and why.
 *  - Unless a parameter says "host", every data pointer is a DEVICE pointer
 *    owned by the caller; the library keeps no reference after the call.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *    Calls are asynchronous on that stream and never synchronise it, except
 *    the *_host entry points, which synchronise the stream before returning.
 *  - The library allocates no device memory.  Calls that need scratch take a
 *    caller workspace (`ws`, `ws_bytes`, 256-byte aligned) whose size is given
 *    by qnn_workspace_bytes(); passing too little returns QNN_ERR_WORKSPACE.
 *  - Leading dimensions are in elements (floats, int32, bytes) or, for packed
 *    data, in 32-bit words.
 *
 * Canonical packed format (crosses the ABI between calls):
 *    row-major uint32_t [rows, ld_words]; element k of a row is bit (k mod 32)
 *    of word (k div 32), least significant bit = lowest k.  Bit 1 means +1
 *    (sign data) or "plane bit set" (bit-plane data).  All pad bits of the
 *    last used word (positions k >= K) are ZERO.  Words at index
 *    >= ceil(K/32) of a row are ignored on input and untouched on output.
 *    A k-bit tensor is `bits` such matrices, `plane_stride_words` apart;
 *    plane i holds bit i of the integer code (i = 0 least significant, the
 *    paper's plane n = i + 1 in Eq. 8).
 *
 * Operand value modes for bit-plane tensors:
 *    QNN_MODE_U01  planes are {0,1}; the value is the unsigned code q = sum_i 2^i p_i
 *    QNN_MODE_PM1  planes are {-1,+1}; the value is sum_i 2^i s_i = 2q - (2^bits - 1)
 */
#ifndef QNN_H_
#define QNN_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define QNN_API __attribute__((visibility("default")))
#else
#define QNN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define QNN_VERSION 230

/* status codes */
#define QNN_OK 0
#define QNN_ERR_INVALID_ARG 1 /* NULL pointer, negative size, bad enum, ld too small      */
#define QNN_ERR_ALIGNMENT 2   /* pointer or leading dimension not aligned as documented   */
#define QNN_ERR_UNSUPPORTED 3 /* valid request this build does not implement              */
#define QNN_ERR_OVERFLOW 4    /* K * max|a| * max|b| does not fit int32                   */
#define QNN_ERR_WORKSPACE 5   /* workspace missing, misaligned or too small               */
#define QNN_ERR_CUDA 6        /* a CUDA runtime call failed (text in qnn_last_error)      */
#define QNN_ERR_TIMEOUT 7     /* a bounded device-side wait ran out (see qnn_device_status) */

/* matrix-product algorithms */
#define QNN_ALGO_AUTO 0   /* library picks per shape                                      */
#define QNN_ALGO_POPC 1   /* xor/and + popc on the CUDA cores (Eq. 11 as written)          */
#define QNN_ALGO_TC_I8 2  /* values expanded to int8, tcgen05 kind::i8, TMEM accumulators */
#define QNN_ALGO_B1_MMA 3 /* 1-bit mma.sync and/xor-popc (legacy tensor-core path)        */
#define QNN_ALGO_TC_FP4 4 /* values as 4-bit e2m1 floats, tcgen05 kind::mxf4 with unit block
                             scales, fp32 TMEM accumulators (exact: integer sums below 2^24);
                             operands of at most 2 planes                                 */

#define QNN_ALGO_TC_PACKED 5 /* the e2m1 product straight from the packed planes: packed tiles by TMA into shared
                             memory, expanded to values there, one launch, NO workspace; operands of at most
                             2 planes, sums below 2^24; 16-byte aligned rows (ld a multiple of 4 words).  What
                             QNN_ALGO_AUTO takes for small batches when it is given no usable workspace   */

/* tensor-core operand forms: one VALUE per element, rows packed along K, pad positions 0 */
#define QNN_FORM_I8 1     /* one byte per element: int8 (QNN_MODE_PM1) or uint8 (QNN_MODE_U01) */
#define QNN_FORM_FP4 2    /* one e2m1 nibble per element, element 2i in the low nibble of byte i;
                             holds the values {0, +-1, +-2, +-3}                            */

#define QNN_MODE_U01 0
#define QNN_MODE_PM1 1

/* operations, for qnn_workspace_bytes */
#define QNN_OP_XNOR_GEMM 1
#define QNN_OP_BITPLANE_GEMM 2
#define QNN_OP_CONV2D 3
#define QNN_OP_MLP 4

QNN_API int qnn_version(void);
QNN_API const char *qnn_status_string(int status);
/* Thread-local description of the last error returned on this thread ("" if none). */
QNN_API const char *qnn_last_error(void);

/* ------------------------------------------------------------------------- */
/* Quantise + pack                                                            */
/* ------------------------------------------------------------------------- */

/* Eq. 1 (deterministic binarisation) + the 32-per-word concatenation of Sec. 6.
 * x: fp32 [rows, K] row-major, leading dimension ldx >= K.
 * out: uint32 [rows, ld_words], ld_words >= ceil(K/32); bit = (x >= 0), so
 * +0.0 and -0.0 give 1 and NaN gives 0.
 * row_popc: optional int32 [rows], receives the number of set bits per row. */
QNN_API int qnn_quantize_pack_sign(const float *x, int64_t rows, int64_t K, int64_t ldx, uint32_t *out,
                           int64_t ld_words, int32_t *row_popc, void *stream);

/* Same binarisation for a weight matrix stored as the paper writes it, W[K, N]
 * row-major (ldw >= N): packs along K for every output unit n, producing
 * out[N, ld_words] -- the "B" operand layout of the matrix products below. */
QNN_API int qnn_quantize_pack_sign_t(const float *w, int64_t K, int64_t N, int64_t ldw, uint32_t *out,
                             int64_t ld_words, int32_t *row_popc, void *stream);

/* Eq. 1 for an NCHW activation tensor x[B,C,H,W] (dense): packs along the
 * channel dimension into out[B,H,W,ceil(C/32)] words (dense NHWC bits), the
 * input layout of qnn_binary_conv2d. */
QNN_API int qnn_quantize_pack_sign_nchw(const float *x, int B, int C, int H, int W, uint32_t *out,
                                void *stream);

/* Eq. 9 read as a uniform quantiser with 2^bits levels on [lo, hi]
 * (bits in 1..8): t = clip(x, lo, hi); code q = round_half_even((t - lo) * inv_step),
 * inv_step = (2^bits - 1) / (hi - lo) evaluated in fp32; all steps are single
 * IEEE fp32 operations (no fused multiply-add).  NaN gives code 0.
 * Writes `bits` planes: planes + i * plane_stride_words is uint32 [rows, ld_words].
 * row_sum_q: optional int32 [rows] = sum_k q[row, k]. */
QNN_API int qnn_quantize_pack_kbit(const float *x, int64_t rows, int64_t K, int64_t ldx, int bits, float lo,
                           float hi, uint32_t *planes, int64_t ld_words, int64_t plane_stride_words,
                           int32_t *row_sum_q, void *stream);

/* Transposed twin for weights W[K, N] row-major: planes are [N, ld_words], packed along K. */
QNN_API int qnn_quantize_pack_kbit_t(const float *w, int64_t K, int64_t N, int64_t ldw, int bits, float lo,
                             float hi, uint32_t *planes, int64_t ld_words, int64_t plane_stride_words,
                             int32_t *row_sum_q, void *stream);

/* Eq. 8 / Algorithm 4 first layer: splits unsigned fixed-point inputs x
 * (uint8 [rows, K], ldx >= K bytes) into their `bits` (1..8) low bit-planes. */
QNN_API int qnn_pack_planes_u8(const uint8_t *x, int64_t rows, int64_t K, int64_t ldx, int bits,
                       uint32_t *planes, int64_t ld_words, int64_t plane_stride_words,
                       int32_t *row_sum_q, void *stream);

/* Section 5 binary convolution weights: w fp32 [Cout, C, KH, KW] (dense) is
 * binarised with Eq. 1 and laid out as out[Cout, KH*KW*ceil(C/32)] words, the
 * reduction ordered (kh, kw, channel word) to match the packed im2col rows. */
QNN_API int qnn_pack_conv_weights(const float *w, int Cout, int C, int KH, int KW, uint32_t *out, void *stream);

/* Table 7, the first fully-connected layer after the last convolution: its
 * inputs are the H x W x C feature map in (h, w, c) order, i.e. the packed NHWC
 * bits of that map read as one row in which every pixel is padded to whole
 * words.  w fp32 [H*W*C, N] row-major (input index (h*W + w)*C + c) is
 * binarised with Eq. 1 and laid out as out[N, H*W*ceil(C/32)] words to match. */
QNN_API int qnn_pack_fc_after_conv_weights(const float *w, int N, int C, int H, int W, uint32_t *out, void *stream);

/* ------------------------------------------------------------------------- */
/* Matrix products                                                            */
/* ------------------------------------------------------------------------- */

/* Algorithm 4 "XnorDotProduct" / Eq. 11:
 * out[m, n] = sum_{k<K} a[m,k] * b[n,k] over +-1 values = K - 2 * popc(a XOR b).
 * a: packed [M, lda], b: packed [N, ldb] (both packed along K, pad bits zero),
 * out: int32 [M, ldo], ldo >= N.  K < 2^31.
 * algo: QNN_ALGO_*; ws/ws_bytes: see qnn_workspace_bytes (may be NULL/0 for POPC). */
QNN_API int qnn_xnor_gemm(const uint32_t *a, int64_t lda, const uint32_t *b, int64_t ldb, int64_t M,
                  int64_t N, int64_t K, int32_t *out, int64_t ldo, int algo, void *ws,
                  size_t ws_bytes, void *stream);

/* The same product with Algorithm 4's Sign(BatchNorm(.)) folded in (see
 * qnn_fold_bn): out_bits[m, n] = (dot[m,n] >= thr[n]) XOR flip[n], packed
 * along n into uint32 [M, ld_words] -- the next layer's "a" operand.
 * thr: int32 [N]; flip: uint8 [N] or NULL (all zero). */
QNN_API int qnn_xnor_gemm_threshold(const uint32_t *a, int64_t lda, const uint32_t *b, int64_t ldb, int64_t M,
                            int64_t N, int64_t K, const int32_t *thr, const uint8_t *flip,
                            uint32_t *out_bits, int64_t ld_words, int algo, void *ws,
                            size_t ws_bytes, void *stream);

/* Eq. 8 generalised (Sec. 3: k-bit operands cost ka*kb binary products):
 * out[m,n] = sum_k A[m,k] * B[n,k], where A, B are the integer values of the
 * ka- and kb-plane tensors under their modes (QNN_MODE_*).
 * a: ka planes of [M, lda], a_plane_stride words apart; b likewise [N, ldb].
 * Requires K * (2^ka - 1) * (2^kb - 1) < 2^31, else QNN_ERR_OVERFLOW. */
QNN_API int qnn_bitplane_gemm(const uint32_t *a, int ka, int a_mode, int64_t lda, int64_t a_plane_stride,
                      const uint32_t *b, int kb, int b_mode, int64_t ldb, int64_t b_plane_stride,
                      int64_t M, int64_t N, int64_t K, int32_t *out, int64_t ldo, int algo, void *ws,
                      size_t ws_bytes, void *stream);

QNN_API int qnn_bitplane_gemm_threshold(const uint32_t *a, int ka, int a_mode, int64_t lda,
                                int64_t a_plane_stride, const uint32_t *b, int kb, int b_mode,
                                int64_t ldb, int64_t b_plane_stride, int64_t M, int64_t N, int64_t K,
                                const int32_t *thr, const uint8_t *flip, uint32_t *out_bits,
                                int64_t ld_words, int algo, void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------- */
/* Tensor-core operands prepared once (static weights, chained layers)        */
/* ------------------------------------------------------------------------- */

/* The tensor-core algorithms multiply VALUES, not bits: each call of the
 * products above first rewrites both packed operands in a tensor-core form in
 * the workspace.  For an operand that does not change between calls (weights)
 * that rewrite can be done once with qnn_tc_prepack and the result handed to
 * qnn_tc_gemm; the thresholded output of qnn_tc_gemm can be produced directly
 * in a form, ready to be the next product's A operand (Algorithm 4 chains
 * a^b_k = Sign(BatchNorm(a_k)) into the next XnorDotProduct).
 *
 * Layout of a form: row-major bytes [rows, ld_bytes]; ld_bytes a multiple of 16
 * and the base 16-byte aligned; a row holds 32 * ceil(K / 32) elements
 * (QNN_FORM_I8: that many bytes; QNN_FORM_FP4: half as many), pad elements 0. */

/* Best form for a product of ka-plane (a_mode) and kb-plane (b_mode) operands
 * over K: QNN_FORM_FP4 when both hold at most 2 planes and K * maxA * maxB < 2^24,
 * else QNN_FORM_I8 when the codes fit a byte, else 0 (use QNN_ALGO_POPC). */
QNN_API int qnn_tc_form(int ka, int a_mode, int kb, int b_mode, int64_t K);

/* Recommended bytes between rows and bytes of a whole operand [rows, K] in `form`:
 * the bytes K elements need (32 * ceil(K / 32) elements: that many bytes in
 * QNN_FORM_I8, half as many in QNN_FORM_FP4) rounded up to whole 128-byte lines.
 * Any multiple of 16 that covers the elements is accepted, but rows that do not
 * start on 128-byte lines make every tile load touch twice the cache lines. */
QNN_API int64_t qnn_tc_row_bytes(int64_t K, int form);
QNN_API size_t qnn_tc_operand_bytes(int64_t rows, int64_t K, int form);

/* Rewrites nplanes packed planes (layout as in qnn_bitplane_gemm) as values in
 * `form`: out[rows, ld_bytes].  QNN_ERR_UNSUPPORTED if the values do not fit. */
QNN_API int qnn_tc_prepack(const uint32_t *planes, int nplanes, int mode, int64_t ld, int64_t plane_stride,
                           int64_t rows, int64_t K, int form, void *out, int64_t ld_bytes, void *stream);

typedef struct qnn_tc_operand {
    const void *data; /* device, form bytes [rows, ld_bytes]                         */
    int64_t ld_bytes;
    int form;         /* QNN_FORM_*                                                  */
    int planes;       /* planes of the integer code the values came from (1..8)      */
    int mode;         /* QNN_MODE_*                                                  */
} qnn_tc_operand;

typedef struct qnn_tc_output { /* any subset; at least one of out / out_bits / out_form */
    int32_t *out;         /* int32 [M, ldo] or NULL                                  */
    int64_t ldo;
    const int32_t *thr;   /* int32 [N], needed for out_bits / out_form               */
    const uint8_t *flip;  /* uint8 [N] or NULL                                       */
    uint32_t *out_bits;   /* packed (dot >= thr) XOR flip, [M, ld_words], or NULL    */
    int64_t ld_words;
    void *out_form;       /* the same signs as +-1 values in form out_form_kind, or NULL */
    int out_form_kind;
    int64_t ld_form_bytes;
} qnn_tc_output;

/* out[m,n] = sum_k A[m,k] * B[n,k] on prepared operands (same form for both).
 * The A operand of a QNN_FORM_I8 product may also be a plain uint8 / int8 matrix
 * of codes (planes = their bit-width) with ld_bytes >= K: Eq. 8's 8-bit input
 * needs no plane split on this path. */
QNN_API int qnn_tc_gemm(const qnn_tc_operand *a, const qnn_tc_operand *b, int64_t M, int64_t N, int64_t K,
                        const qnn_tc_output *o, void *stream);

/* Eq. 1 / Eq. 9 straight into a tensor-core form: the same values and layout
 * qnn_quantize_pack_* followed by qnn_tc_prepack would give, in one pass over
 * the fp32 data (4 bytes read, 1/2 or 1 byte written per element, nothing
 * re-read).  out: rows ld_bytes apart (a multiple of 16 covering
 * qnn_tc_row_bytes' element bytes; whole 128-byte lines recommended), 16-byte
 * aligned; elements between K and the next multiple of 32 are written as 0,
 * bytes beyond that are left untouched.
 *   _sign       x [rows, K] row-major              -> +-1 per element
 *   _sign_t     w [K, N] row-major (weights)       -> rows n = 0..N-1 along K
 *   _sign_nchw  x [B, C, H, W]                     -> rows (b, y, x) along C
 *   _kbit / _kbit_t  Eq. 9 codes on [lo, hi]: the code q (mode QNN_MODE_U01)
 *               or 2q - (2^bits - 1) (QNN_MODE_PM1); bits <= 2 for
 *               QNN_FORM_FP4, <= 8 (U01) / 7 (PM1) for QNN_FORM_I8. */
QNN_API int qnn_quantize_form_sign(const float *x, int64_t rows, int64_t K, int64_t ldx, int form, void *out,
                                   int64_t ld_bytes, void *stream);
QNN_API int qnn_quantize_form_sign_t(const float *w, int64_t K, int64_t N, int64_t ldw, int form, void *out,
                                     int64_t ld_bytes, void *stream);
QNN_API int qnn_quantize_form_sign_nchw(const float *x, int B, int C, int H, int W, int form, void *out,
                                        int64_t ld_bytes, void *stream);
QNN_API int qnn_quantize_form_kbit(const float *x, int64_t rows, int64_t K, int64_t ldx, int bits, float lo, float hi,
                                   int mode, int form, void *out, int64_t ld_bytes, void *stream);
QNN_API int qnn_quantize_form_kbit_t(const float *w, int64_t K, int64_t N, int64_t ldw, int bits, float lo, float hi,
                                     int mode, int form, void *out, int64_t ld_bytes, void *stream);

/* Algorithm 4's hidden-layer product for a SMALL batch whose weights are still
 * real-valued, in one pass over them:
 *   out[m, n] = sum_k sign(x[m, k]) * sign(w[k, n])      (Eq. 1 on both operands)
 * x fp32 [M, K] (ldx), w fp32 [K, N] row-major (ldw), out int32 [M, ldo].
 * The kernel binarises the weights while it streams them (4 bytes per weight,
 * read once, nothing packed is written or re-read) and multiplies on the
 * tensor cores; the result equals qnn_quantize_pack_sign + _sign_t +
 * qnn_xnor_gemm bit for bit.  Meant for M up to a few hundred rows: every
 * further 128 rows of the batch stream the weights again.  K < 2^24.
 * ws: qnn_fc_sign_f32_workspace_bytes(M, K) bytes (the activations as values). */
QNN_API size_t qnn_fc_sign_f32_workspace_bytes(int64_t M, int64_t K);
QNN_API int qnn_fc_sign_f32(const float *x, int64_t M, int64_t K, int64_t ldx, const float *w, int64_t N, int64_t ldw,
                            int32_t *out, int64_t ldo, void *ws, size_t ws_bytes, void *stream);

/* Size of the scratch array built into the library for qnn_xnor_gemm_noalloc. */
#define QNN_NOALLOC_SCRATCH_BYTES (8u << 20)

/* The paper has no counterpart for this call; it is a packaging variant of
 * qnn_xnor_gemm (same arguments, same int32 result, always the int8 tensor-core
 * algorithm) for callers that cannot allocate device memory or size a
 * workspace when they call: code running on a latency-critical serving thread
 * where cudaMalloc's implicit device synchronisation would stall every stream,
 * plug-ins that are handed only their input and output buffers by a host
 * framework that owns the allocator, and processes whose whole memory budget
 * was reserved up front so that a later cudaMalloc simply fails.
 *
 * The int8 operand scratch is a fixed QNN_NOALLOC_SCRATCH_BYTES (8 MiB) array
 * inside the library image: every GPU context that loads the library holds it
 * until the process exits.  The call performs no cudaMalloc / cudaFree and
 * calls no allocating library routine.  Shapes whose scratch
 *   (M + N) * roundup(32 * ceil(K / 32), 128)   bytes (the M and the N term each rounded up to 256)
 * exceeds the array are rejected with QNN_ERR_WORKSPACE before anything runs
 * (e.g. 1024 x 1024 x 4096 fits, 4096 x 4096 x 4096 does not).
 *
 * The first call on each device looks up the array's device address (a
 * one-time host-side set-up under a mutex, with that device current); make
 * that first call before starting any stream capture.  All calls share the one
 * array, which keeps the previous call's contents: the call rewrites every
 * byte it later reads, so no clearing is needed, but two calls that overlap on
 * the GPU (different streams, or several host threads) race on it -- keep
 * calls to this entry point on one stream or serialise them yourself.
 * K = 0 gives all zeros like qnn_xnor_gemm.  The looked-up address is kept for
 * the life of the process and does not survive cudaDeviceReset: do not call
 * this entry point on a device after resetting it. */
QNN_API int qnn_xnor_gemm_noalloc(const uint32_t *a, int64_t lda, const uint32_t *b, int64_t ldb, int64_t M,
                                  int64_t N, int64_t K, int32_t *out, int64_t ldo, void *stream);

/* ------------------------------------------------------------------------- */
/* Threshold, rescale                                                         */
/* ------------------------------------------------------------------------- */

/* Algorithm 4, a^b = Sign(BatchNorm(a)): standalone form on an int32 matrix
 * s[M, lds]: out[m, n] = (s[m,n] >= thr[n]) XOR flip[n], packed along n. */
QNN_API int qnn_threshold_pack(const int32_t *s, int64_t M, int64_t N, int64_t lds, const int32_t *thr,
                       const uint8_t *flip, uint32_t *out, int64_t ld_words, void *stream);

/* HOST helper (host pointers, no GPU work): folds inference-time batch norm
 * y = gamma * (s - mean) / sqrt(var + eps) + beta followed by Eq. 1 (y >= 0)
 * into integers, in double precision:
 *   gamma > 0: thr = ceil(tau),      flip = 0,  tau = mean - beta * sigma / gamma
 *   gamma < 0: thr = floor(tau) + 1, flip = 1
 *   gamma = 0: thr = INT32_MIN,      flip = (beta < 0)
 * thr is clamped to the int32 range. */
QNN_API int qnn_fold_bn(const double *gamma, const double *beta, const double *mean, const double *var,
                double eps, int64_t N, int32_t *thr_host, uint8_t *flip_host);

/* Algorithm 4 output layer (affine batch norm of the integer scores) and
 * de-quantisation of affine codes:
 * y[m,n] = alpha * p[m,n] + row_off[m] + col_off[n] + delta in fp32
 * (row_off, col_off optional).  Evaluated as ((alpha*p + row) + col) + delta
 * with separate roundings. */
QNN_API int qnn_rescale_f32(const int32_t *p, int64_t M, int64_t N, int64_t ldp, float alpha,
                    const float *row_off, const float *col_off, float delta, float *y, int64_t ldy,
                    void *stream);

/* ------------------------------------------------------------------------- */
/* Binary convolution                                                         */
/* ------------------------------------------------------------------------- */

/* Section 5: out[b,co,y,x] = sum_{c,kh,kw} X[b,c,y*stride+kh-pad,x*stride+kw-pad] * Wt[co,c,kh,kw]
 * over +-1 values (cross-correlation); a tap outside the image reads +1 when
 * pad_bit = 1, -1 when pad_bit = 0.
 * x: packed NHWC bits [B,H,W,ceil(C/32)] (qnn_quantize_pack_sign_nchw);
 * w: [Cout, KH*KW*ceil(C/32)] (qnn_pack_conv_weights).
 * Outputs (either may be NULL, not both): out_nchw int32 [B,Cout,Ho,Wo];
 * out_bits packed NHWC [B,Ho,Wo,ceil(Cout/32)] = (out >= thr[co]) XOR flip[co]
 * (thr required when out_bits is given).
 * The packed im2col matrix [B*Ho*Wo, KH*KW*ceil(C/32)] lives in the workspace. */
QNN_API int qnn_binary_conv2d(const uint32_t *x, int B, int C, int H, int W, const uint32_t *w, int Cout,
                      int KH, int KW, int stride, int pad, int pad_bit, int32_t *out_nchw,
                      const int32_t *thr, const uint8_t *flip, uint32_t *out_bits, int algo, void *ws,
                      size_t ws_bytes, void *stream);

/* Filter banks prepared once (static weights) for the tensor-core convolution.
 * Applies to stride-1 "same" filters (KH = KW = 2 * pad + 1, at most 7 x 7) with
 * C a multiple of 128 and images at most 128 pixels wide; qnn_conv_form(C) is the
 * form such a layer multiplies in (QNN_FORM_FP4: a pixel is 128-byte channel
 * blocks when C % 256 == 0, else 64-byte ones; 0 = not available: use
 * qnn_binary_conv2d).
 * qnn_conv_prepare rewrites w (qnn_pack_conv_weights layout) in that form and
 * appends the table of what the padding value contributes per border position;
 * `prepared` is a 256-byte aligned device buffer of qnn_conv_prepared_bytes. */
QNN_API int qnn_conv_form(int C);
QNN_API size_t qnn_conv_prepared_bytes(int Cout, int C, int KH, int KW, int pad);
QNN_API int qnn_conv_prepare(const uint32_t *w, int Cout, int C, int KH, int KW, int pad, int pad_bit,
                             void *prepared, size_t prepared_bytes, void *stream);

typedef struct qnn_conv_io {
    const void *x;        /* x_form 0: packed NHWC bits [B,H,W,ceil(C/32)] words;
                             x_form = qnn_conv_form(C): NHWC values in that form, pixels
                             32*ceil(C/32) elements apart (dense)                        */
    int x_form;
    int32_t *out_nchw;    /* int32 [B,Cout,H,W] or NULL                                  */
    const int32_t *thr;   /* int32 [Cout], needed for out_bits / out_form               */
    const uint8_t *flip;  /* uint8 [Cout] or NULL                                        */
    uint32_t *out_bits;   /* packed NHWC bits [B,H,W,ceil(Cout/32)] or NULL              */
    void *out_form;       /* the same signs as NHWC values in out_form_kind (dense), the
                             next convolution's x, or NULL                               */
    int out_form_kind;
    int pool2x2;          /* 1: 2 x 2 max-pooling between the convolution and the threshold
                             (Table 7), done inside the call on the thresholded signs:
                             out_bits / out_form are then [B, H/2, W/2, ...]; needs
                             qnn_conv_can_pool(H, W) and out_nchw == NULL                */
} qnn_conv_io;

/* 1 when qnn_binary_conv2d_prepared can pool inside the call: W in {2,4,8,16} and H even
 * (a window's four pixels then sit in one warp of the epilogue); other sizes pool with
 * qnn_maxpool2x2_bits. */
QNN_API int qnn_conv_can_pool(int H, int W);

/* Section 5 with a prepared filter bank: same result as qnn_binary_conv2d
 * (stride 1, the pad and pad_bit given to qnn_conv_prepare).  A workspace of
 * B*H*W * 32*ceil(C/32) bytes (int8 form; half for e2m1) is needed only when x is
 * given as packed bits. */
QNN_API int qnn_binary_conv2d_prepared(const qnn_conv_io *io, int B, int C, int H, int W, const void *prepared,
                                       int Cout, int KH, int KW, int pad, void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------- */
/* Algorithm 4 runner                                                         */
/* ------------------------------------------------------------------------- */

/* One layer of the MLP (a HOST struct; the pointers inside are device pointers). */
typedef struct qnn_mlp_layer {
    const uint32_t *w;   /* packed weights [N, ldw], packed along K           */
    int64_t ldw;         /* words                                             */
    int64_t K;           /* inputs of this layer                              */
    int64_t N;           /* units of this layer                               */
    const int32_t *thr;  /* int32 [N]; ignored for the last layer             */
    const uint8_t *flip; /* uint8 [N] or NULL; ignored for the last layer     */
    /* Optional: the same weights already in a tensor-core form (qnn_tc_prepack
     * with 1 plane, QNN_MODE_PM1), so that the runner does not rewrite them on
     * every pass.  Used when w_tc != NULL and w_tc_form is the form the layer
     * runs in (qnn_mlp_layer_form); ignored otherwise. */
    const void *w_tc;
    int64_t w_tc_ld;     /* bytes between rows of w_tc                        */
    int w_tc_form;       /* QNN_FORM_*                                        */
} qnn_mlp_layer;

/* Form in which layer `l` multiplies when it runs on the tensor cores
 * (layer 0: in_bits-bit unsigned codes x +-1 weights; others +-1 x +-1). */
QNN_API int qnn_mlp_layer_form(const qnn_mlp_layer *layers, int L, int l, int in_bits);

/* Algorithm 4 "Running a BNN with L layers" on device buffers:
 * layer 1 is the bit-plane product of the in_bits-bit input (Eq. 8), hidden
 * layers are XNOR products with folded thresholds, the last layer returns
 * int32 scores[M, layers[L-1].N] (its affine batch norm is qnn_rescale_f32).
 * x: uint8 [M, layers[0].K] dense.  layers: HOST array of L structs. */
QNN_API int qnn_mlp_forward(const uint8_t *x, int64_t M, int in_bits, const qnn_mlp_layer *layers, int L,
                    int32_t *scores, int algo, void *ws, size_t ws_bytes, void *stream);

/* Same, for callers holding HOST buffers: copies x_host (pinned memory
 * recommended) to the device, runs the layers, copies the scores back to
 * scores_host and synchronises `stream`.  Batch rows are independent, so large
 * batches are cut into 2 chunks whose input copies (on a copy stream the
 * library creates once per device and keeps) overlap the previous chunk's
 * layers; the copies start after the work already queued on `stream`.  The
 * workspace must also hold the input and the scores: size it with
 * qnn_mlp_workspace_bytes(..., 1). */
QNN_API int qnn_mlp_forward_host(const uint8_t *x_host, int64_t M, int in_bits, const qnn_mlp_layer *layers,
                         int L, int32_t *scores_host, int algo, void *ws, size_t ws_bytes,
                         void *stream);

/* The same pass from HOST buffers as one CUDA graph (Algorithm 4 end to end:
 * input copies, every layer, the copy of the scores back).  _create runs the
 * pass once, captures a second issue of it on `stream` (which must not be the
 * default stream) and instantiates the graph; _launch replays it with one
 * launch, asynchronously on the given stream -- synchronise that stream before
 * reading scores_host.  The graph refers to x_host, scores_host (both must be
 * pinned host memory and stay valid), the layers' buffers and ws as they were
 * at creation: write new inputs into the same x_host buffer between launches.
 * chunks (1..8): pieces the batch is cut into so that input copies overlap the
 * previous piece's layers; with the launch overhead gone, 3-4 pays for large
 * batches.  The handle is a small host object the caller owns; the library
 * allocates no device memory for it (the CUDA runtime keeps the graph). */
typedef struct qnn_mlp_graph qnn_mlp_graph;
QNN_API int qnn_mlp_graph_create(const uint8_t *x_host, int64_t M, int in_bits, const qnn_mlp_layer *layers, int L,
                                 int32_t *scores_host, int algo, void *ws, size_t ws_bytes, int chunks, void *stream,
                                 qnn_mlp_graph **out);
QNN_API int qnn_mlp_graph_launch(qnn_mlp_graph *g, void *stream);
QNN_API int qnn_mlp_graph_destroy(qnn_mlp_graph *g);

QNN_API size_t qnn_mlp_workspace_bytes(int64_t M, int in_bits, const qnn_mlp_layer *layers, int L, int algo,
                               int host_io);

/* Logarithmic quantiser, Eq. 10: LogQuant(x) = Clip(AP2(x), minV, maxV) with
 * AP2(x) = sign(x) * 2^round(log2|x|) (caption of Algorithm 2), the magnitude
 * clipped to minV = 2^emin ... maxV = 2^emax.  Each element is written as the
 * int8 value sign * 2^(e - emin), e = clamp(round(log2|x|), emin, emax): the
 * quantised value in units of minV, which is an operand of the int8 tensor-core
 * form as it stands (qnn_tc_gemm with form QNN_FORM_I8, mode QNN_MODE_PM1 and
 * planes = emax - emin + 1, so that |value| <= 2^planes - 1); the product of two such
 * matrices is the exact integer sum in units of minV_a * minV_b.
 * Rounding: log2|x| has no ties on floats (sqrt(2) is not a float); zero and
 * denormals clip to emin, infinities and NaN to emax; sign as in Eq. 1.
 *   x    device, float [rows, ldx]
 *   out  device, int8 [rows, ld_bytes], ld_bytes >= K rounded up to 32 and a
 *        multiple of 4 (of 16 to serve as a tensor-core operand); bytes K ...
 *        roundup(K, 32) of every row are written as zero
 * Errors: INVALID_ARG, UNSUPPORTED (emax - emin > 6: 2^7 does not fit int8),
 * ALIGNMENT, CUDA. */
QNN_API int qnn_logquant_pack_i8(const float *x, int64_t rows, int64_t K, int64_t ldx, int emin, int emax, void *out,
                                 int64_t ld_bytes, void *stream);

/* Eq. 10 with up to 31 exponents (a 6-bit code: a sign and 5 bits of exponent), for the
 * backward products of Algorithm 1 with quantised gradients (Sec. 4.4: of the gradient
 * quantisers tried only the logarithmic one worked, at 6 bits; end of Sec. 5: quantised
 * gradients let the backward pass use the binary kernel): gradient x +-1 weights, and +-1 activations x gradient.
 * A code sign * 2^(e - emin) with e - emin up to 30 has one set bit; the exponents are cut
 * into groups of seven, group g holding sign * 2^(e - emin - 7g) where e falls into it and
 * 0 elsewhere.  qnn_logquant_groups = the number of groups G = (emax - emin) / 7 + 1
 * (0 when the range is not 0..30).  qnn_logquant_pack_groups writes the G group matrices
 * stacked row-wise, int8 [G * rows, ld_bytes] (group g at rows g*rows ..): ONE operand of
 * the int8 tensor-core form (qnn_tc_gemm, QNN_FORM_I8, QNN_MODE_PM1, 7 planes) whose
 * product with a +-1 matrix is int32 [G * rows, N]; qnn_logquant_combine then gives
 *     out[m, n] = sum_g 2^(7g) * p[g * M + m, n]
 * the exact sum of code x weight in int64, in units of 2^emin.
 *   x           device, float; transposed = 0: [rows, ldx], a row of x is a row of the
 *               operand (K elements); transposed = 1: [K, ldx >= rows], a COLUMN of x is a
 *               row of the operand (the weight gradient contracts over the batch)
 *   out         device, int8 [G * rows, ld_bytes]; ld_bytes >= K rounded up to 32, a multiple
 *               of 4 (of 16 to serve as a tensor-core operand); bytes K .. roundup(K, 32) of
 *               every row are written as zero
 *   p, out(i64) device; ldp, ldo in elements
 * Rounding, zero, infinities, NaN and the sign as in qnn_logquant_pack_i8.
 * Errors: INVALID_ARG, UNSUPPORTED (more than 31 exponents), ALIGNMENT, CUDA. */
QNN_API int qnn_logquant_groups(int emin, int emax);
QNN_API int qnn_logquant_pack_groups(const float *x, int64_t rows, int64_t K, int64_t ldx, int transposed, int emin, int emax,
                                     void *out, int64_t ld_bytes, void *stream);
QNN_API int qnn_logquant_combine(const int32_t *p, int groups, int64_t M, int64_t N, int64_t ldp, int64_t *out, int64_t ldo,
                                 void *stream);

/* ------------------------------------------------------------------------- */
/* The ConvNet of Table 7                                                     */
/* ------------------------------------------------------------------------- */

/* First layer of Table 7: a stride-1 convolution of 8-bit pixel codes with +-1
 * filters, i.e. Eq. 8 summed over the eight bit planes:
 *   out[b,co,y,x] = sum_{c,kh,kw} q[b,c,y+kh-pad,x+kw-pad] * w[co,c,kh,kw],
 * a tap outside the image reading pad_code (0 = the zero border of a 'same'
 * convolution).  Runs as an im2col of the codes and one int8 tensor-core product.
 *   x         device, uint8 [B,C,H,W]
 *   w         device, packed filters as qnn_pack_conv_weights writes them
 *   out_nchw  device, int32 [B,Cout,Ho,Wo] or NULL (Ho = H + 2 pad - KH + 1)
 *   thr/flip  folded batch norm, needed for out_bits / out_form
 *   out_bits  device, packed NHWC bits [B,Ho,Wo,ceil(Cout/32)] or NULL
 *   out_form  device, the same signs as NHWC values in out_form_kind
 *             (QNN_FORM_*; pixels 32*ceil(Cout/32) elements apart), or NULL
 *   ws        256-byte aligned scratch of qnn_conv2d_u8_workspace_bytes(...)
 * Errors: INVALID_ARG, UNSUPPORTED (KH*KW*C > 8192), WORKSPACE, CUDA. */
QNN_API size_t qnn_conv2d_u8_workspace_bytes(int B, int C, int H, int W, int Cout, int KH, int KW, int pad);
QNN_API int qnn_conv2d_u8(const uint8_t *x, int B, int C, int H, int W, const uint32_t *w, int Cout, int KH, int KW,
                          int pad, int pad_code, int32_t *out_nchw, const int32_t *thr, const uint8_t *flip,
                          uint32_t *out_bits, void *out_form, int out_form_kind, void *ws, size_t ws_bytes,
                          void *stream);

/* 2 x 2 / stride 2 max-pooling placed between a convolution and its batch norm
 * (Table 7), applied AFTER the folded threshold: since the threshold is
 * monotone in the sum, the bit of a window's largest sum is the OR of its four
 * bits, and the AND for channels with flip[c] != 0.  A trailing odd row or
 * column is dropped.
 *   bits      device, packed NHWC bits [B,H,W,ceil(C/32)] (pad bits zero)
 *   flip      device, uint8 [C] (the flip given to the threshold) or NULL
 *   out_bits  device, [B,H/2,W/2,ceil(C/32)] or NULL
 *   out_form  device, the pooled signs as NHWC values in out_form_kind, or NULL */
QNN_API int qnn_maxpool2x2_bits(const uint32_t *bits, int B, int H, int W, int C, const uint8_t *flip,
                                uint32_t *out_bits, void *out_form, int out_form_kind, void *stream);

#define QNN_LAYER_CONV_U8 1 /* first layer: 8-bit codes x +-1 filters, zero border        */
#define QNN_LAYER_CONV 2    /* +-1 x +-1 'same' convolution, border value +1              */
#define QNN_LAYER_FC 3      /* fully connected +-1 x +-1                                   */

/* One layer of a ConvNet (a HOST struct; the pointers inside are device pointers). */
typedef struct qnn_net_layer {
    int kind;            /* QNN_LAYER_*                                                     */
    int C;               /* convolution: input channels; FC: inputs                        */
    int Cout;            /* convolution: output channels; FC: units                        */
    int ksize;           /* convolution: ksize x ksize filter, ksize = 2 * pad + 1         */
    int pad;
    int pool;            /* convolution: 1 = 2 x 2 max-pooling before the threshold        */
    const uint32_t *w;   /* convolution: qnn_pack_conv_weights layout [Cout, k*k*ceil(C/32)];
                            FC after a convolution: the same layout for a [Cout, C', H', W']
                            filter covering the whole feature map (inputs in (h, w, c)
                            order, each pixel padded to whole words); FC after an FC layer:
                            [Cout, ceil(C/32)]                                              */
    const int32_t *thr;  /* int32 [Cout]; NULL only on the last layer                      */
    const uint8_t *flip; /* uint8 [Cout] or NULL                                           */
} qnn_net_layer;

/* Table 7 at inference, layer by layer on one stream: convolution, optional
 * pooling, folded batch norm + binarisation (Algorithm 4's a^b), then the fully
 * connected layers; the last layer (FC) returns int32 scores [B, Cout].
 * Convolutions with C a multiple of 128 and images up to 128 wide run as
 * implicit products on the tensor cores from filter banks prepared once by
 * qnn_convnet_prepare (activations pass between them in tensor-core form);
 * other shapes take the packed im2col path.
 *   x         device, uint8 [B, layers[0].C, H, W]
 *   prepared  device, written by qnn_convnet_prepare for the same layers, H, W
 *   ws        256-byte aligned scratch of qnn_convnet_workspace_bytes(...)
 * Errors: INVALID_ARG (layers that do not chain), UNSUPPORTED, WORKSPACE, CUDA. */
QNN_API size_t qnn_convnet_prepared_bytes(int H, int W, const qnn_net_layer *layers, int n);
QNN_API int qnn_convnet_prepare(int H, int W, const qnn_net_layer *layers, int n, void *prepared,
                                size_t prepared_bytes, void *stream);
QNN_API size_t qnn_convnet_workspace_bytes(int B, int H, int W, const qnn_net_layer *layers, int n);
QNN_API int qnn_convnet_forward(const uint8_t *x, int B, int H, int W, const qnn_net_layer *layers, int n,
                                const void *prepared, int32_t *scores, void *ws, size_t ws_bytes, void *stream);

/* ------------------------------------------------------------------------- */
/* Workspace, status                                                          */
/* ------------------------------------------------------------------------- */

/* Scratch bytes for one call of `op` (QNN_OP_XNOR_GEMM, QNN_OP_BITPLANE_GEMM:
 * M,N,K,ka,kb; QNN_OP_CONV2D: M = B*Ho*Wo, N = Cout, K = KH*KW*32*ceil(C/32),
 * ka = kb = 1) under `algo`.  0 means no workspace is needed. */
QNN_API size_t qnn_workspace_bytes(int op, int64_t M, int64_t N, int64_t K, int ka, int kb, int algo);

/* Which algorithm QNN_ALGO_AUTO resolves to for a shape (never returns AUTO). */
QNN_API int qnn_select_algo(int64_t M, int64_t N, int64_t K, int ka, int kb, int a_mode, int b_mode);

/* Tensor-core kernels bound every device-side wait; when one runs out the
 * kernel records it in a per-process device status word and exits cleanly.
 * This call synchronises `stream`, reads and clears that word and returns
 * QNN_OK or QNN_ERR_TIMEOUT. */
QNN_API int qnn_device_status(void *stream);

/* Diagnostic (the paper has no counterpart): launches one tiny kernel whose
 * only action is a bounded wait, with a limit of a few thousand polls, on a
 * barrier that nothing arrives on -- no copy and no tensor-core work is in
 * flight.  The wait runs out through the same code the product kernels use,
 * so the next qnn_device_status() returns QNN_ERR_TIMEOUT once and QNN_OK
 * after that, and the context stays fully usable.  For checking the failure
 * path of an installation; never needed in normal operation. */
QNN_API int qnn_selftest_wait_timeout(void *stream);

/* Measurement aid: arms two cudaEvent_t handles (passed as void*) on the calling
 * thread.  The next matrix-product call made by this thread records `start`
 * immediately before and `stop` immediately after its product kernel (not
 * around operand expansion or im2col), on that call's stream, and disarms
 * them.  Pass NULLs to disarm. */
QNN_API int qnn_set_kernel_events(void *start, void *stop);

/* Same, but the events go around the (nth + 1)-th matrix-product kernel this thread launches from now on
 * (nth = 0 is the next one): lets one layer inside qnn_mlp_forward be timed. */
QNN_API int qnn_set_kernel_events_nth(void *start, void *stop, int nth);

/* Measurement aid (the paper has no counterpart): launches one kernel that
 * keeps a pipe busy with nothing else in the way -- every SM multiplies one
 * resident shared-memory tile pair `iters` times with the tensor-core
 * instruction the product kernels use (128 x 256 x 32 bytes of K, e2m1 with
 * unit block scales or int8; no loads, no epilogue), or runs Eq. 11's xor /
 * popc / add on registers.  *ops_host receives the operations one launch
 * performs (2 per multiply-accumulate; 64 per 32-bit xor/popc/add); the caller
 * times the launch with its own events.  The product kernels' speed is quoted
 * against these figures as well as against the library-GEMM proxy. */
#define QNN_PIPE_TENSOR_FP4 1
#define QNN_PIPE_TENSOR_I8 2
#define QNN_PIPE_POPC 3
QNN_API int qnn_pipe_peak_launch(int pipe, int iters, double *ops_host, void *stream);

/* Number of kernels this library has launched in this process so far (all
 * threads, all streams); a monotonically increasing bookkeeping counter. */
QNN_API uint64_t qnn_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* QNN_H_ */
