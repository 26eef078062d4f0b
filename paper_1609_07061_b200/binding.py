"""ctypes binding of libqnn.so: argument marshalling only.

Every function mirrors the C entry point of the same name (see include/qnn.h).
Tensors are torch CUDA tensors; the binding passes their data pointers, sizes
and the current CUDA stream, raises ``QnnError`` on a non-zero status and does
no arithmetic of its own.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqnn.so")

QNN_OK = 0
QNN_ERR_INVALID_ARG, QNN_ERR_ALIGNMENT, QNN_ERR_UNSUPPORTED, QNN_ERR_OVERFLOW = 1, 2, 3, 4
QNN_ERR_WORKSPACE, QNN_ERR_CUDA, QNN_ERR_TIMEOUT = 5, 6, 7
QNN_ALGO_AUTO, QNN_ALGO_POPC, QNN_ALGO_TC_I8, QNN_ALGO_B1_MMA, QNN_ALGO_TC_FP4, QNN_ALGO_TC_PACKED = 0, 1, 2, 3, 4, 5
QNN_FORM_I8, QNN_FORM_FP4 = 1, 2
QNN_MODE_U01, QNN_MODE_PM1 = 0, 1
QNN_OP_XNOR_GEMM, QNN_OP_BITPLANE_GEMM, QNN_OP_CONV2D, QNN_OP_MLP = 1, 2, 3, 4
QNN_LAYER_CONV_U8, QNN_LAYER_CONV, QNN_LAYER_FC = 1, 2, 3
QNN_NOALLOC_SCRATCH_BYTES = 8 << 20


class QnnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({_lib.qnn_status_string(status).decode()}): "
                         f"{_lib.qnn_last_error().decode()}")


if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_1609_07061_b200.build` "
        "(nvcc, sm_100a).  There is no CPU fallback.")

_lib = ctypes.CDLL(LIB_PATH)

i64, i32, vp, f32, sz = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_float, ctypes.c_size_t


class qnn_tc_operand(ctypes.Structure):
    _fields_ = [("data", vp), ("ld_bytes", i64), ("form", i32), ("planes", i32), ("mode", i32)]


class qnn_tc_output(ctypes.Structure):
    _fields_ = [("out", vp), ("ldo", i64), ("thr", vp), ("flip", vp), ("out_bits", vp), ("ld_words", i64),
                ("out_form", vp), ("out_form_kind", i32), ("ld_form_bytes", i64)]


class qnn_conv_io(ctypes.Structure):
    _fields_ = [("x", vp), ("x_form", i32), ("out_nchw", vp), ("thr", vp), ("flip", vp), ("out_bits", vp),
                ("out_form", vp), ("out_form_kind", i32), ("pool2x2", i32)]


class qnn_mlp_layer(ctypes.Structure):
    _fields_ = [("w", vp), ("ldw", i64), ("K", i64), ("N", i64), ("thr", vp), ("flip", vp),
                ("w_tc", vp), ("w_tc_ld", i64), ("w_tc_form", i32)]


class qnn_net_layer(ctypes.Structure):
    _fields_ = [("kind", i32), ("C", i32), ("Cout", i32), ("ksize", i32), ("pad", i32), ("pool", i32),
                ("w", vp), ("thr", vp), ("flip", vp)]


_SIGS = {
    "qnn_version": (i32, []),
    "qnn_status_string": (ctypes.c_char_p, [i32]),
    "qnn_last_error": (ctypes.c_char_p, []),
    "qnn_quantize_pack_sign": (i32, [vp, i64, i64, i64, vp, i64, vp, vp]),
    "qnn_quantize_pack_sign_t": (i32, [vp, i64, i64, i64, vp, i64, vp, vp]),
    "qnn_quantize_pack_sign_nchw": (i32, [vp, i32, i32, i32, i32, vp, vp]),
    "qnn_quantize_pack_kbit": (i32, [vp, i64, i64, i64, i32, f32, f32, vp, i64, i64, vp, vp]),
    "qnn_quantize_pack_kbit_t": (i32, [vp, i64, i64, i64, i32, f32, f32, vp, i64, i64, vp, vp]),
    "qnn_pack_planes_u8": (i32, [vp, i64, i64, i64, i32, vp, i64, i64, vp, vp]),
    "qnn_pack_conv_weights": (i32, [vp, i32, i32, i32, i32, vp, vp]),
    "qnn_pack_fc_after_conv_weights": (i32, [vp, i32, i32, i32, i32, vp, vp]),
    "qnn_xnor_gemm": (i32, [vp, i64, vp, i64, i64, i64, i64, vp, i64, i32, vp, sz, vp]),
    "qnn_xnor_gemm_noalloc": (i32, [vp, i64, vp, i64, i64, i64, i64, vp, i64, vp]),
    "qnn_xnor_gemm_threshold": (i32, [vp, i64, vp, i64, i64, i64, i64, vp, vp, vp, i64, i32, vp, sz, vp]),
    "qnn_bitplane_gemm": (i32, [vp, i32, i32, i64, i64, vp, i32, i32, i64, i64, i64, i64, i64, vp, i64, i32, vp, sz, vp]),
    "qnn_bitplane_gemm_threshold": (i32, [vp, i32, i32, i64, i64, vp, i32, i32, i64, i64, i64, i64, i64, vp, vp, vp,
                                          i64, i32, vp, sz, vp]),
    "qnn_quantize_form_sign": (i32, [vp, i64, i64, i64, i32, vp, i64, vp]),
    "qnn_quantize_form_sign_t": (i32, [vp, i64, i64, i64, i32, vp, i64, vp]),
    "qnn_quantize_form_sign_nchw": (i32, [vp, i32, i32, i32, i32, i32, vp, i64, vp]),
    "qnn_quantize_form_kbit": (i32, [vp, i64, i64, i64, i32, ctypes.c_float, ctypes.c_float, i32, i32, vp, i64, vp]),
    "qnn_quantize_form_kbit_t": (i32, [vp, i64, i64, i64, i32, ctypes.c_float, ctypes.c_float, i32, i32, vp, i64, vp]),
    "qnn_fc_sign_f32_workspace_bytes": (sz, [i64, i64]),
    "qnn_fc_sign_f32": (i32, [vp, i64, i64, i64, vp, i64, i64, vp, i64, vp, sz, vp]),
    "qnn_tc_form": (i32, [i32, i32, i32, i32, i64]),
    "qnn_tc_row_bytes": (i64, [i64, i32]),
    "qnn_tc_operand_bytes": (sz, [i64, i64, i32]),
    "qnn_tc_prepack": (i32, [vp, i32, i32, i64, i64, i64, i64, i32, vp, i64, vp]),
    "qnn_tc_gemm": (i32, [ctypes.POINTER(qnn_tc_operand), ctypes.POINTER(qnn_tc_operand), i64, i64, i64,
                          ctypes.POINTER(qnn_tc_output), vp]),
    "qnn_threshold_pack": (i32, [vp, i64, i64, i64, vp, vp, vp, i64, vp]),
    "qnn_fold_bn": (i32, [vp, vp, vp, vp, ctypes.c_double, i64, vp, vp]),
    "qnn_rescale_f32": (i32, [vp, i64, i64, i64, f32, vp, vp, f32, vp, i64, vp]),
    "qnn_binary_conv2d": (i32, [vp, i32, i32, i32, i32, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, i32, vp, sz, vp]),
    "qnn_conv_form": (i32, [i32]),
    "qnn_conv_can_pool": (i32, [i32, i32]),
    "qnn_conv_prepared_bytes": (sz, [i32, i32, i32, i32, i32]),
    "qnn_logquant_groups": (i32, [i32, i32]),
    "qnn_logquant_pack_groups": (i32, [vp, i64, i64, i64, i32, i32, i32, vp, i64, vp]),
    "qnn_logquant_combine": (i32, [vp, i32, i64, i64, i64, vp, i64, vp]),
    "qnn_conv_prepare": (i32, [vp, i32, i32, i32, i32, i32, i32, vp, sz, vp]),
    "qnn_binary_conv2d_prepared": (i32, [ctypes.POINTER(qnn_conv_io), i32, i32, i32, i32, vp, i32, i32, i32, i32, vp, sz, vp]),
    "qnn_logquant_pack_i8": (i32, [vp, i64, i64, i64, i32, i32, vp, i64, vp]),
    "qnn_conv2d_u8_workspace_bytes": (sz, [i32, i32, i32, i32, i32, i32, i32, i32]),
    "qnn_conv2d_u8": (i32, [vp, i32, i32, i32, i32, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32, vp, sz, vp]),
    "qnn_maxpool2x2_bits": (i32, [vp, i32, i32, i32, i32, vp, vp, vp, i32, vp]),
    "qnn_convnet_prepared_bytes": (sz, [i32, i32, ctypes.POINTER(qnn_net_layer), i32]),
    "qnn_convnet_prepare": (i32, [i32, i32, ctypes.POINTER(qnn_net_layer), i32, vp, sz, vp]),
    "qnn_convnet_workspace_bytes": (sz, [i32, i32, i32, ctypes.POINTER(qnn_net_layer), i32]),
    "qnn_convnet_forward": (i32, [vp, i32, i32, i32, ctypes.POINTER(qnn_net_layer), i32, vp, vp, vp, sz, vp]),
    "qnn_mlp_forward": (i32, [vp, i64, i32, ctypes.POINTER(qnn_mlp_layer), i32, vp, i32, vp, sz, vp]),
    "qnn_mlp_forward_host": (i32, [vp, i64, i32, ctypes.POINTER(qnn_mlp_layer), i32, vp, i32, vp, sz, vp]),
    "qnn_mlp_graph_create": (i32, [vp, i64, i32, ctypes.POINTER(qnn_mlp_layer), i32, vp, i32, vp, sz, i32, vp, ctypes.POINTER(vp)]),
    "qnn_mlp_graph_launch": (i32, [vp, vp]),
    "qnn_mlp_graph_destroy": (i32, [vp]),
    "qnn_mlp_layer_form": (i32, [ctypes.POINTER(qnn_mlp_layer), i32, i32, i32]),
    "qnn_mlp_workspace_bytes": (sz, [i64, i32, ctypes.POINTER(qnn_mlp_layer), i32, i32, i32]),
    "qnn_workspace_bytes": (sz, [i32, i64, i64, i64, i32, i32, i32]),
    "qnn_select_algo": (i32, [i64, i64, i64, i32, i32, i32, i32]),
    "qnn_device_status": (i32, [vp]),
    "qnn_selftest_wait_timeout": (i32, [vp]),
    "qnn_pipe_peak_launch": (i32, [i32, i32, ctypes.POINTER(ctypes.c_double), vp]),
    "qnn_launch_count": (ctypes.c_uint64, []),
    "qnn_set_kernel_events": (i32, [vp, vp]),
    "qnn_set_kernel_events_nth": (i32, [vp, vp, i32]),
}
for _name, (_res, _args) in _SIGS.items():
    _fn = getattr(_lib, _name)          # AttributeError here = the library does not export a declared symbol
    _fn.restype = _res
    _fn.argtypes = _args

EXPORTED = tuple(_SIGS.keys())


def _p(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream():
    # without a CUDA device only host-side validation can succeed; any launch then returns QNN_ERR_CUDA
    return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None


def _ck(status: int, where: str):
    if status != QNN_OK:
        raise QnnError(status, where)


def _ws(ws: Optional[torch.Tensor]):
    return (None, 0) if ws is None else (ws.data_ptr(), ws.numel() * ws.element_size())


def qnn_version() -> int:
    return _lib.qnn_version()


def qnn_status_string(status: int) -> str:
    return _lib.qnn_status_string(status).decode()


def qnn_last_error() -> str:
    return _lib.qnn_last_error().decode()


def qnn_quantize_pack_sign(x, rows, K, ldx, out, ld_words, row_popc=None):
    _ck(_lib.qnn_quantize_pack_sign(_p(x), rows, K, ldx, _p(out), ld_words, _p(row_popc), _stream()),
        "qnn_quantize_pack_sign")


def qnn_quantize_pack_sign_t(w, K, N, ldw, out, ld_words, row_popc=None):
    _ck(_lib.qnn_quantize_pack_sign_t(_p(w), K, N, ldw, _p(out), ld_words, _p(row_popc), _stream()),
        "qnn_quantize_pack_sign_t")


def qnn_quantize_pack_sign_nchw(x, B, C, H, W, out):
    _ck(_lib.qnn_quantize_pack_sign_nchw(_p(x), B, C, H, W, _p(out), _stream()), "qnn_quantize_pack_sign_nchw")


def qnn_quantize_pack_kbit(x, rows, K, ldx, bits, lo, hi, planes, ld_words, plane_stride_words, row_sum_q=None):
    _ck(_lib.qnn_quantize_pack_kbit(_p(x), rows, K, ldx, bits, lo, hi, _p(planes), ld_words, plane_stride_words,
                                    _p(row_sum_q), _stream()), "qnn_quantize_pack_kbit")


def qnn_quantize_pack_kbit_t(w, K, N, ldw, bits, lo, hi, planes, ld_words, plane_stride_words, row_sum_q=None):
    _ck(_lib.qnn_quantize_pack_kbit_t(_p(w), K, N, ldw, bits, lo, hi, _p(planes), ld_words, plane_stride_words,
                                      _p(row_sum_q), _stream()), "qnn_quantize_pack_kbit_t")


def qnn_pack_planes_u8(x, rows, K, ldx, bits, planes, ld_words, plane_stride_words, row_sum_q=None):
    _ck(_lib.qnn_pack_planes_u8(_p(x), rows, K, ldx, bits, _p(planes), ld_words, plane_stride_words, _p(row_sum_q),
                                _stream()), "qnn_pack_planes_u8")


def qnn_pack_conv_weights(w, Cout, C, KH, KW, out):
    _ck(_lib.qnn_pack_conv_weights(_p(w), Cout, C, KH, KW, _p(out), _stream()), "qnn_pack_conv_weights")


def qnn_pack_fc_after_conv_weights(w, N, C, H, W, out):
    _ck(_lib.qnn_pack_fc_after_conv_weights(_p(w), N, C, H, W, _p(out), _stream()), "qnn_pack_fc_after_conv_weights")


def qnn_xnor_gemm(a, lda, b, ldb, M, N, K, out, ldo, algo=QNN_ALGO_AUTO, ws=None):
    wp, wb = _ws(ws)
    _ck(_lib.qnn_xnor_gemm(_p(a), lda, _p(b), ldb, M, N, K, _p(out), ldo, algo, wp, wb, _stream()), "qnn_xnor_gemm")


def qnn_xnor_gemm_threshold(a, lda, b, ldb, M, N, K, thr, flip, out_bits, ld_words, algo=QNN_ALGO_AUTO, ws=None):
    wp, wb = _ws(ws)
    _ck(_lib.qnn_xnor_gemm_threshold(_p(a), lda, _p(b), ldb, M, N, K, _p(thr), _p(flip), _p(out_bits), ld_words, algo,
                                     wp, wb, _stream()), "qnn_xnor_gemm_threshold")


def qnn_bitplane_gemm(a, ka, a_mode, lda, a_plane_stride, b, kb, b_mode, ldb, b_plane_stride, M, N, K, out, ldo,
                      algo=QNN_ALGO_AUTO, ws=None):
    wp, wb = _ws(ws)
    _ck(_lib.qnn_bitplane_gemm(_p(a), ka, a_mode, lda, a_plane_stride, _p(b), kb, b_mode, ldb, b_plane_stride, M, N, K,
                               _p(out), ldo, algo, wp, wb, _stream()), "qnn_bitplane_gemm")


def qnn_bitplane_gemm_threshold(a, ka, a_mode, lda, a_plane_stride, b, kb, b_mode, ldb, b_plane_stride, M, N, K, thr,
                                flip, out_bits, ld_words, algo=QNN_ALGO_AUTO, ws=None):
    wp, wb = _ws(ws)
    _ck(_lib.qnn_bitplane_gemm_threshold(_p(a), ka, a_mode, lda, a_plane_stride, _p(b), kb, b_mode, ldb,
                                         b_plane_stride, M, N, K, _p(thr), _p(flip), _p(out_bits), ld_words, algo, wp,
                                         wb, _stream()), "qnn_bitplane_gemm_threshold")


def qnn_tc_form(ka, a_mode, kb, b_mode, K) -> int:
    return int(_lib.qnn_tc_form(ka, a_mode, kb, b_mode, K))


def qnn_tc_row_bytes(K, form) -> int:
    return int(_lib.qnn_tc_row_bytes(K, form))


def qnn_tc_operand_bytes(rows, K, form) -> int:
    return int(_lib.qnn_tc_operand_bytes(rows, K, form))


def qnn_tc_prepack(planes, nplanes, mode, ld, plane_stride, rows, K, form, out, ld_bytes):
    _ck(_lib.qnn_tc_prepack(_p(planes), nplanes, mode, ld, plane_stride, rows, K, form, _p(out), ld_bytes, _stream()),
        "qnn_tc_prepack")


def qnn_quantize_form_sign(x, rows, K, ldx, form, out, ld_bytes):
    _ck(_lib.qnn_quantize_form_sign(_p(x), rows, K, ldx, form, _p(out), ld_bytes, _stream()), "qnn_quantize_form_sign")


def qnn_quantize_form_sign_t(w, K, N, ldw, form, out, ld_bytes):
    _ck(_lib.qnn_quantize_form_sign_t(_p(w), K, N, ldw, form, _p(out), ld_bytes, _stream()), "qnn_quantize_form_sign_t")


def qnn_quantize_form_sign_nchw(x, B, C, H, W, form, out, ld_bytes):
    _ck(_lib.qnn_quantize_form_sign_nchw(_p(x), B, C, H, W, form, _p(out), ld_bytes, _stream()), "qnn_quantize_form_sign_nchw")


def qnn_quantize_form_kbit(x, rows, K, ldx, bits, lo, hi, mode, form, out, ld_bytes):
    _ck(_lib.qnn_quantize_form_kbit(_p(x), rows, K, ldx, bits, lo, hi, mode, form, _p(out), ld_bytes, _stream()),
        "qnn_quantize_form_kbit")


def qnn_quantize_form_kbit_t(w, K, N, ldw, bits, lo, hi, mode, form, out, ld_bytes):
    _ck(_lib.qnn_quantize_form_kbit_t(_p(w), K, N, ldw, bits, lo, hi, mode, form, _p(out), ld_bytes, _stream()),
        "qnn_quantize_form_kbit_t")


def qnn_fc_sign_f32_workspace_bytes(M, K) -> int:
    return int(_lib.qnn_fc_sign_f32_workspace_bytes(M, K))


def qnn_fc_sign_f32(x, M, K, ldx, w, N, ldw, out, ldo, ws):
    """out = sign(x) . sign(w) from fp32 activations [M, K] and fp32 weights [K, N], weights read once (small batches)."""
    wp, wb = _ws(ws)
    _ck(_lib.qnn_fc_sign_f32(_p(x), M, K, ldx, _p(w), N, ldw, _p(out), ldo, wp, wb, _stream()), "qnn_fc_sign_f32")


def tc_operand(data, ld_bytes, form, planes=1, mode=QNN_MODE_PM1) -> qnn_tc_operand:
    return qnn_tc_operand(_p(data), ld_bytes, form, planes, mode)


def qnn_tc_gemm(a: qnn_tc_operand, b: qnn_tc_operand, M, N, K, out=None, ldo=0, thr=None, flip=None, out_bits=None,
                ld_words=0, out_form=None, out_form_kind=0, ld_form_bytes=0):
    o = qnn_tc_output(_p(out), ldo, _p(thr), _p(flip), _p(out_bits), ld_words, _p(out_form), out_form_kind,
                      ld_form_bytes)
    _ck(_lib.qnn_tc_gemm(ctypes.byref(a), ctypes.byref(b), M, N, K, ctypes.byref(o), _stream()), "qnn_tc_gemm")


def qnn_threshold_pack(s, M, N, lds, thr, flip, out, ld_words):
    _ck(_lib.qnn_threshold_pack(_p(s), M, N, lds, _p(thr), _p(flip), _p(out), ld_words, _stream()),
        "qnn_threshold_pack")


def qnn_fold_bn(gamma, beta, mean, var, eps, thr_host, flip_host):
    """All arguments are CPU tensors (float64 in, int32 / uint8 out)."""
    N = gamma.numel()
    _ck(_lib.qnn_fold_bn(_p(gamma), _p(beta), _p(mean), _p(var), float(eps), N, _p(thr_host), _p(flip_host)),
        "qnn_fold_bn")


def qnn_rescale_f32(p, M, N, ldp, alpha, row_off, col_off, delta, y, ldy):
    _ck(_lib.qnn_rescale_f32(_p(p), M, N, ldp, alpha, _p(row_off), _p(col_off), delta, _p(y), ldy, _stream()),
        "qnn_rescale_f32")


def qnn_binary_conv2d(x, B, C, H, W, w, Cout, KH, KW, stride, pad, pad_bit, out_nchw, thr, flip, out_bits,
                      algo=QNN_ALGO_AUTO, ws=None):
    wp, wb = _ws(ws)
    _ck(_lib.qnn_binary_conv2d(_p(x), B, C, H, W, _p(w), Cout, KH, KW, stride, pad, pad_bit, _p(out_nchw), _p(thr),
                               _p(flip), _p(out_bits), algo, wp, wb, _stream()), "qnn_binary_conv2d")


def qnn_conv_form(C) -> int:
    return int(_lib.qnn_conv_form(C))


def qnn_logquant_groups(emin, emax) -> int:
    return int(_lib.qnn_logquant_groups(emin, emax))


def qnn_logquant_pack_groups(x, rows, K, ldx, transposed, emin, emax, out, ld_bytes):
    _ck(_lib.qnn_logquant_pack_groups(_p(x), rows, K, ldx, int(transposed), emin, emax, _p(out), ld_bytes, _stream()),
        "qnn_logquant_pack_groups")


def qnn_logquant_combine(p, groups, M, N, ldp, out, ldo):
    _ck(_lib.qnn_logquant_combine(_p(p), groups, M, N, ldp, _p(out), ldo, _stream()), "qnn_logquant_combine")


def qnn_conv_prepared_bytes(Cout, C, KH, KW, pad) -> int:
    return int(_lib.qnn_conv_prepared_bytes(Cout, C, KH, KW, pad))


def qnn_conv_prepare(w, Cout, C, KH, KW, pad, pad_bit, prepared):
    _ck(_lib.qnn_conv_prepare(_p(w), Cout, C, KH, KW, pad, pad_bit, _p(prepared), prepared.numel() * prepared.element_size(),
                              _stream()), "qnn_conv_prepare")


def qnn_binary_conv2d_prepared(x, x_form, B, C, H, W, prepared, Cout, KH, KW, pad, out_nchw=None, thr=None, flip=None,
                               out_bits=None, out_form=None, out_form_kind=0, ws=None, pool2x2=0):
    io = qnn_conv_io(_p(x), x_form, _p(out_nchw), _p(thr), _p(flip), _p(out_bits), _p(out_form), out_form_kind, pool2x2)
    wp, wb = _ws(ws)
    _ck(_lib.qnn_binary_conv2d_prepared(ctypes.byref(io), B, C, H, W, _p(prepared), Cout, KH, KW, pad, wp, wb, _stream()),
        "qnn_binary_conv2d_prepared")


def make_mlp_layers(ws: Sequence[torch.Tensor], ldws: Sequence[int], Ks: Sequence[int], Ns: Sequence[int],
                    thrs: Sequence[Optional[torch.Tensor]], flips: Sequence[Optional[torch.Tensor]]):
    """Builds the host array of qnn_mlp_layer structs (pointer marshalling only)."""
    L = len(ws)
    arr = (qnn_mlp_layer * L)()
    for l in range(L):
        arr[l].w = _p(ws[l])
        arr[l].ldw = ldws[l]
        arr[l].K = Ks[l]
        arr[l].N = Ns[l]
        arr[l].thr = _p(thrs[l]) if l < len(thrs) else None
        arr[l].flip = _p(flips[l]) if l < len(flips) else None
    return arr


def qnn_mlp_layer_form(layers, l, in_bits) -> int:
    return int(_lib.qnn_mlp_layer_form(layers, len(layers), l, in_bits))


def prepack_mlp_weights(layers, ws: Sequence[torch.Tensor], in_bits: int) -> List[torch.Tensor]:
    """Rewrites every layer's packed weights once in the tensor-core form the layer runs in (qnn_tc_prepack) and
    stores the pointers in the layer structs.  Returns the buffers: the caller keeps them alive."""
    keep = []
    for l in range(len(layers)):
        form = qnn_mlp_layer_form(layers, l, in_bits)
        if form == 0:
            continue
        K, N = int(layers[l].K), int(layers[l].N)
        rb = qnn_tc_row_bytes(K, form)
        buf = torch.empty(N, rb, dtype=torch.uint8, device="cuda")
        qnn_tc_prepack(ws[l], 1, QNN_MODE_PM1, int(layers[l].ldw), 0, N, K, form, buf, rb)
        layers[l].w_tc, layers[l].w_tc_ld, layers[l].w_tc_form = buf.data_ptr(), rb, form
        keep.append(buf)
    return keep


def qnn_mlp_workspace_bytes(M, in_bits, layers, algo=QNN_ALGO_AUTO, host_io=0) -> int:
    return int(_lib.qnn_mlp_workspace_bytes(M, in_bits, layers, len(layers), algo, host_io))


def qnn_mlp_forward(x, M, in_bits, layers, scores, algo=QNN_ALGO_AUTO, ws=None):
    wp, wb = _ws(ws)
    _ck(_lib.qnn_mlp_forward(_p(x), M, in_bits, layers, len(layers), _p(scores), algo, wp, wb, _stream()),
        "qnn_mlp_forward")


def qnn_mlp_forward_host(x_host, M, in_bits, layers, scores_host, algo=QNN_ALGO_AUTO, ws=None):
    wp, wb = _ws(ws)
    _ck(_lib.qnn_mlp_forward_host(_p(x_host), M, in_bits, layers, len(layers), _p(scores_host), algo, wp, wb,
                                  _stream()), "qnn_mlp_forward_host")


class MlpGraph:
    """One Algorithm-4 pass from pinned host buffers as a CUDA graph (argument marshalling only)."""

    def __init__(self, x_host, M, in_bits, layers, scores_host, algo, ws, chunks=3):
        wp, wb = _ws(ws)
        self.handle = vp()
        self.keep = (x_host, scores_host, layers, ws)
        self.stream = torch.cuda.Stream()
        self.stream.wait_stream(torch.cuda.current_stream())
        _ck(_lib.qnn_mlp_graph_create(_p(x_host), M, in_bits, layers, len(layers), _p(scores_host), algo, wp, wb, chunks,
                                      self.stream.cuda_stream, ctypes.byref(self.handle)), "qnn_mlp_graph_create")

    def launch(self):
        _ck(_lib.qnn_mlp_graph_launch(self.handle, _stream()), "qnn_mlp_graph_launch")

    def close(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.qnn_mlp_graph_destroy(self.handle)
        self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:       # interpreter shutdown: the library may already be gone
            pass


def qnn_logquant_pack_i8(x, rows, K, ldx, emin, emax, out, ld_bytes):
    _ck(_lib.qnn_logquant_pack_i8(_p(x), rows, K, ldx, emin, emax, _p(out), ld_bytes, _stream()), "qnn_logquant_pack_i8")


def qnn_conv_can_pool(H, W) -> bool:
    return bool(_lib.qnn_conv_can_pool(H, W))


def qnn_conv2d_u8_workspace_bytes(B, C, H, W, Cout, KH, KW, pad) -> int:
    return int(_lib.qnn_conv2d_u8_workspace_bytes(B, C, H, W, Cout, KH, KW, pad))


def qnn_conv2d_u8(x, B, C, H, W, w, Cout, KH, KW, pad, pad_code=0, out_nchw=None, thr=None, flip=None, out_bits=None,
                  out_form=None, out_form_kind=0, ws=None):
    wp, wb = _ws(ws)
    _ck(_lib.qnn_conv2d_u8(_p(x), B, C, H, W, _p(w), Cout, KH, KW, pad, pad_code, _p(out_nchw), _p(thr), _p(flip),
                           _p(out_bits), _p(out_form), out_form_kind, wp, wb, _stream()), "qnn_conv2d_u8")


def qnn_maxpool2x2_bits(bits, B, H, W, C, flip=None, out_bits=None, out_form=None, out_form_kind=0):
    _ck(_lib.qnn_maxpool2x2_bits(_p(bits), B, H, W, C, _p(flip), _p(out_bits), _p(out_form), out_form_kind, _stream()),
        "qnn_maxpool2x2_bits")


def make_net_layers(specs):
    """specs: dicts with kind, C, Cout, and (conv) ksize, pad, pool; w, thr, flip device tensors (thr None on the last)."""
    arr = (qnn_net_layer * len(specs))()
    for i, sp in enumerate(specs):
        arr[i].kind = sp["kind"]
        arr[i].C = sp["C"]
        arr[i].Cout = sp["Cout"]
        arr[i].ksize = sp.get("ksize", 0)
        arr[i].pad = sp.get("pad", 0)
        arr[i].pool = 1 if sp.get("pool") else 0
        arr[i].w = _p(sp["w"])
        arr[i].thr = _p(sp.get("thr"))
        arr[i].flip = _p(sp.get("flip"))
    return arr


class ConvNet:
    """A Table 7 network on the device: packed weights, layer structs, prepared filter banks (argument marshalling only)."""

    def __init__(self, in_ch, H, W, conv_W, conv_pool, fc_W, Ts, flips):
        """conv_W: fp32 [Cout,C,k,k] tensors; fc_W: fp32 [K,N], the first with K in (h, w, c) order of the last
        feature map; Ts / flips: per layer but the last (flips may hold None)."""
        self.H, self.W = H, W
        self.keep, specs = [], []
        c, h, w, t = in_ch, H, W, 0
        for i, (Wc, pool) in enumerate(zip(conv_W, conv_pool)):
            co, ci, k, _ = Wc.shape
            wb = torch.zeros(co, k * k * ((ci + 31) // 32), dtype=torch.int32, device="cuda")
            qnn_pack_conv_weights(Wc.cuda().contiguous(), co, ci, k, k, wb)
            specs.append(dict(kind=QNN_LAYER_CONV_U8 if i == 0 else QNN_LAYER_CONV, C=ci, Cout=co, ksize=k, pad=k // 2,
                              pool=pool, w=wb, thr=Ts[t].cuda(), flip=None if flips[t] is None else flips[t].cuda()))
            t += 1
            c = co
            if pool:
                h, w = h // 2, w // 2
        first = True
        for j, Wf in enumerate(fc_W):
            K, N = Wf.shape
            last = j == len(fc_W) - 1
            if first and len(conv_W) > 0:
                # inputs in (h, w, c) order, every pixel padded to whole words
                wb = torch.zeros(N, h * w * ((c + 31) // 32), dtype=torch.int32, device="cuda")
                qnn_pack_fc_after_conv_weights(Wf.cuda().contiguous(), N, c, h, w, wb)
            else:
                ld = (K + 31) // 32
                wb = torch.zeros(N, ld, dtype=torch.int32, device="cuda")
                qnn_quantize_pack_sign_t(Wf.cuda().contiguous(), K, N, N, wb, ld)
            first = False
            specs.append(dict(kind=QNN_LAYER_FC, C=K, Cout=N, w=wb, thr=None if last else Ts[t].cuda(),
                              flip=None if (last or flips[t] is None) else flips[t].cuda()))
            t += 0 if last else 1
        self.n_out = specs[-1]["Cout"]
        self.keep = specs
        self.layers = make_net_layers(specs)
        nb = qnn_convnet_prepared_bytes(H, W, self.layers)
        if nb == 0:
            raise QnnError(QNN_ERR_INVALID_ARG, "qnn_convnet_prepared_bytes")
        self.prepared = torch.empty(nb, dtype=torch.uint8, device="cuda")
        qnn_convnet_prepare(H, W, self.layers, self.prepared)

    def workspace(self, B) -> torch.Tensor:
        nb = qnn_convnet_workspace_bytes(B, self.H, self.W, self.layers)
        if nb == 0 and B > 0:
            raise QnnError(QNN_ERR_INVALID_ARG, "qnn_convnet_workspace_bytes")
        return torch.empty(max(nb, 256), dtype=torch.uint8, device="cuda")

    def forward(self, x, scores, ws):
        qnn_convnet_forward(x, x.shape[0], self.H, self.W, self.layers, self.prepared, scores, ws)


def qnn_convnet_prepared_bytes(H, W, layers) -> int:
    return int(_lib.qnn_convnet_prepared_bytes(H, W, layers, len(layers)))


def qnn_convnet_prepare(H, W, layers, prepared):
    _ck(_lib.qnn_convnet_prepare(H, W, layers, len(layers), _p(prepared), prepared.numel() * prepared.element_size(), _stream()),
        "qnn_convnet_prepare")


def qnn_convnet_workspace_bytes(B, H, W, layers) -> int:
    return int(_lib.qnn_convnet_workspace_bytes(B, H, W, layers, len(layers)))


def qnn_convnet_forward(x, B, H, W, layers, prepared, scores, ws=None):
    wp, wb = _ws(ws)
    _ck(_lib.qnn_convnet_forward(_p(x), B, H, W, layers, len(layers), _p(prepared), _p(scores), wp, wb, _stream()),
        "qnn_convnet_forward")


def qnn_workspace_bytes(op, M, N, K, ka=1, kb=1, algo=QNN_ALGO_AUTO) -> int:
    return int(_lib.qnn_workspace_bytes(op, M, N, K, ka, kb, algo))


def qnn_select_algo(M, N, K, ka=1, kb=1, a_mode=QNN_MODE_PM1, b_mode=QNN_MODE_PM1) -> int:
    return int(_lib.qnn_select_algo(M, N, K, ka, kb, a_mode, b_mode))


def qnn_device_status() -> int:
    return int(_lib.qnn_device_status(_stream()))


def qnn_selftest_wait_timeout():
    """Launches the diagnostic kernel whose bounded wait runs out; the next qnn_device_status() reports it once."""
    _ck(_lib.qnn_selftest_wait_timeout(_stream()), "qnn_selftest_wait_timeout")


QNN_PIPE_TENSOR_FP4, QNN_PIPE_TENSOR_I8, QNN_PIPE_POPC = 1, 2, 3


def qnn_pipe_peak_launch(pipe: int, iters: int) -> float:
    """Launches the issue-only measurement kernel of `pipe`; returns the operations that launch performs."""
    ops = ctypes.c_double(0.0)
    _ck(_lib.qnn_pipe_peak_launch(pipe, iters, ctypes.byref(ops), _stream()), "qnn_pipe_peak_launch")
    return float(ops.value)


def qnn_launch_count() -> int:
    return int(_lib.qnn_launch_count())


def qnn_set_kernel_events(start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]):
    """Arms two torch CUDA events (already created, i.e. recorded once) around the next product kernel."""
    a = None if start is None else start.cuda_event
    b = None if stop is None else stop.cuda_event
    _ck(_lib.qnn_set_kernel_events(a, b), "qnn_set_kernel_events")


def qnn_set_kernel_events_nth(start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event], nth: int):
    """As qnn_set_kernel_events, around the (nth + 1)-th product kernel launched from now on."""
    a = None if start is None else start.cuda_event
    b = None if stop is None else stop.cuda_event
    _ck(_lib.qnn_set_kernel_events_nth(a, b, nth), "qnn_set_kernel_events_nth")


def qnn_xnor_gemm_noalloc(a, lda, b, ldb, M, N, K, out, ldo):
    """XNOR product whose scratch is the library's built-in 8 MiB array: no workspace argument, no allocation.

    For callers that cannot allocate device memory at call time.  Calls share the array, so keep them on one
    stream; the first call on a device should precede any stream capture."""
    _ck(_lib.qnn_xnor_gemm_noalloc(_p(a), lda, _p(b), ldb, M, N, K, _p(out), ldo, _stream()), "qnn_xnor_gemm_noalloc")
