"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, validates arguments
before launching, and its host helpers (batch-norm fold, workspace sizing) behave."""
import os
import re

import numpy as np
import pytest
import torch

import oracle


@pytest.fixture(scope="module")
def q():
    import __graft_entry__ as ge
    ge.build()
    import paper_1609_07061_b200.binding as b
    return b


ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_symbol_is_exported(q):
    hdr = open(os.path.join(ROOT, "include", "qnn.h")).read()
    declared = set(re.findall(r"QNN_API\s+[\w\s\*]+?\b(qnn_\w+)\s*\(", hdr))
    assert len(declared) >= 24
    for name in declared:
        assert hasattr(q._lib, name), f"{name} declared in qnn.h but not exported by libqnn.so"
    assert declared == set(q.EXPORTED), declared ^ set(q.EXPORTED)


def test_version_and_strings(q):
    assert q.qnn_version() == 230
    assert q.qnn_status_string(0) == "ok"
    assert "overflow" in q.qnn_status_string(q.QNN_ERR_OVERFLOW)


def test_validation_errors_without_launch(q):
    fake = torch.zeros(64, dtype=torch.int32)          # CPU memory: never dereferenced, validation fails first
    with pytest.raises(q.QnnError) as e:
        q.qnn_xnor_gemm(fake, 1, fake, 1, 4, 4, -1, fake, 4)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as e:               # lda smaller than ceil(K/32)
        q.qnn_xnor_gemm(fake, 1, fake, 2, 4, 4, 64, fake, 4)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as e:               # ldo < N
        q.qnn_xnor_gemm(fake, 2, fake, 2, 4, 4, 64, fake, 3)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as e:               # 8b x 8b with K = 2^20 overflows int32
        q.qnn_bitplane_gemm(fake, 8, 0, 1 << 15, 1 << 30, fake, 8, 0, 1 << 15, 1 << 30, 4, 4, 1 << 20, fake, 4)
    assert e.value.status == q.QNN_ERR_OVERFLOW
    with pytest.raises(q.QnnError) as e:
        q.qnn_quantize_pack_kbit(fake, 2, 8, 8, 9, 0.0, 1.0, fake, 1, 2)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as e:
        q.qnn_quantize_pack_kbit(fake, 2, 8, 8, 2, 1.0, 1.0, fake, 1, 2)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as e:               # conv without workspace
        q.qnn_binary_conv2d(fake, 1, 32, 4, 4, fake, 8, 3, 3, 1, 1, 1, fake, None, None, None)
    assert e.value.status == q.QNN_ERR_WORKSPACE
    with pytest.raises(q.QnnError) as e:               # bits output without thresholds
        q.qnn_xnor_gemm_threshold(fake, 2, fake, 2, 4, 4, 64, None, None, fake, 1)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    assert q.qnn_last_error() != ""


def test_empty_shapes_are_ok(q):
    q.qnn_xnor_gemm(None, 0, None, 0, 0, 0, 0, None, 0)
    q.qnn_quantize_pack_sign(None, 0, 16, 16, None, 1)
    q.qnn_threshold_pack(None, 0, 8, 8, None, None, None, 1)


def test_fold_bn_matches_direct_batch_norm(q):
    """Folded integer threshold == double-precision BN + sign on every integer pre-activation in [-K, K]."""
    rng = np.random.default_rng(0)
    K = 300
    s = np.arange(-K, K + 1, dtype=np.int32)
    N = 64
    gamma = rng.standard_normal(N)
    gamma[:4] = [0.0, 0.0, 1e-3, -1e-3]
    beta = rng.standard_normal(N) * 3
    beta[0], beta[1] = 0.5, -0.5
    mean = rng.standard_normal(N) * 40 + 0.123          # irrational-ish offsets keep tau away from integers
    var = rng.uniform(0.5, 400.0, N)
    eps = 1e-4
    thr = torch.empty(N, dtype=torch.int32)
    flip = torch.empty(N, dtype=torch.uint8)
    q.qnn_fold_bn(torch.from_numpy(gamma), torch.from_numpy(beta), torch.from_numpy(mean), torch.from_numpy(var), eps,
                  thr, flip)
    for n in range(N):
        sigma = float(np.sqrt(var[n] + eps))
        want = oracle.bn_sign_direct(s, gamma[n], beta[n], mean[n], sigma)
        got = oracle.threshold(s.reshape(-1, 1), thr[n:n + 1].numpy(), flip[n:n + 1].numpy()).reshape(-1)
        # exact ties of the real-valued BN (y == 0 up to rounding) are excluded: not claimed
        tau = mean[n] - beta[n] * sigma / gamma[n] if gamma[n] != 0 else None
        keep = np.ones_like(s, bool) if tau is None else np.abs(s - tau) > 1e-6
        np.testing.assert_array_equal(got[keep], want[keep], err_msg=f"channel {n}")
    assert thr[0].item() == -2**31 and flip[0].item() == 0 and flip[1].item() == 1


def test_workspace_sizes(q):
    assert q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, 128, 128, 1024, 1, 1, q.QNN_ALGO_POPC) == 0
    conv = q.qnn_workspace_bytes(q.QNN_OP_CONV2D, 128 * 16 * 16, 256, 9 * 256, 1, 1, q.QNN_ALGO_POPC)
    assert conv >= 128 * 16 * 16 * 72 * 4
    layers = q.make_mlp_layers([torch.zeros(1, dtype=torch.int32)] * 2, [25, 128], [784, 4096], [4096, 10],
                               [torch.zeros(1, dtype=torch.int32)], [None])
    assert q.qnn_mlp_workspace_bytes(100, 8, layers, q.QNN_ALGO_POPC, 0) > 100 * 28 * 4 * 8
    assert q.qnn_mlp_workspace_bytes(100, 8, layers, q.QNN_ALGO_POPC, 1) > q.qnn_mlp_workspace_bytes(
        100, 8, layers, q.QNN_ALGO_POPC, 0)
