"""GPU test of qnn_xnor_gemm_noalloc, the entry point for callers that cannot allocate device memory
(its operand scratch is an 8 MiB array built into the library).  Collected last on purpose.

It must give exactly what qnn_xnor_gemm gives (integer outputs: bit-exact), on two calls in a row that
share the built-in scratch, whether this file runs alone in a fresh process or after every other test."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def q():
    import paper_1609_07061_b200.binding as b
    return b


def _operands(M, N, K, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    kw = (K + 31) // 32
    ld = (kw + 3) // 4 * 4
    a = torch.randint(-2**31, 2**31 - 1, (M, ld), dtype=torch.int32, device="cuda", generator=g)
    b = torch.randint(-2**31, 2**31 - 1, (N, ld), dtype=torch.int32, device="cuda", generator=g)
    if K % 32:                                   # the packed format wants zero pad bits in the last used word
        mask = (1 << (K % 32)) - 1
        m32 = mask if mask < 2**31 else mask - 2**32
        a[:, kw - 1] &= m32
        b[:, kw - 1] &= m32
    return a, b, ld


def test_noalloc_matches_workspace_entry_point_twice_in_a_row(q):
    # second call: other shape, other data, smaller K -- stale scratch from the first call must not leak in
    for (M, N, K, seed) in [(300, 1000, 4096, 1), (257, 130, 1000, 2)]:
        a, b, ld = _operands(M, N, K, seed)
        want = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
        ws = torch.empty(max(q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, q.QNN_ALGO_TC_I8), 256),
                         dtype=torch.uint8, device="cuda")
        q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, want, N, q.QNN_ALGO_TC_I8, ws)
        popc = torch.empty_like(want)
        q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, popc, N, q.QNN_ALGO_POPC)
        got = torch.full((M, N), -9, dtype=torch.int32, device="cuda")
        q.qnn_xnor_gemm_noalloc(a, ld, b, ld, M, N, K, got, N)
        torch.cuda.synchronize()
        assert q.qnn_device_status() == 0
        assert torch.equal(got, want)
        assert torch.equal(got, popc)


def test_noalloc_matches_the_oracle_on_unpacked_bits(q):
    """Parity proper: random 0/1 bits packed by the test's own packer, the product through the no-workspace entry
    point, against the oracle's +-1 matrix product on the unpacked values (and K = 0, an empty sum)."""
    import oracle
    from util import as_i32_words, pack_bits_ref
    rng = np.random.default_rng(11)
    for (M, N, K) in [(130, 70, 1000), (64, 33, 31), (5, 300, 4096)]:
        abits = rng.integers(0, 2, (M, K)).astype(np.uint8)
        bbits = rng.integers(0, 2, (N, K)).astype(np.uint8)
        ld = ((K + 31) // 32 + 3) // 4 * 4
        a = as_i32_words(pack_bits_ref(abits, ld)).cuda()
        b = as_i32_words(pack_bits_ref(bbits, ld)).cuda()
        got = torch.full((M, N), -9, dtype=torch.int32, device="cuda")
        q.qnn_xnor_gemm_noalloc(a, ld, b, ld, M, N, K, got, N)
        torch.cuda.synchronize()
        assert q.qnn_device_status() == 0
        # oracle.xnor_gemm takes real values and applies Eq. 1 itself: feed it +-1 as floats
        want = oracle.xnor_gemm(2.0 * abits.astype(np.float32) - 1.0, (2.0 * bbits.astype(np.float32) - 1.0).T.copy())
        np.testing.assert_array_equal(got.cpu().numpy(), want)
    got = torch.full((7, 9), -9, dtype=torch.int32, device="cuda")
    z = torch.zeros(16, 4, dtype=torch.int32, device="cuda")
    q.qnn_xnor_gemm_noalloc(z, 4, z, 4, 7, 9, 0, got, 9)
    torch.cuda.synchronize()
    assert bool((got == 0).all())


def test_noalloc_takes_no_device_memory_and_fits_its_documented_limit(q):
    """1024 x 1024 x 4096 needs exactly the built-in 8 MiB; after the one-time set-up a call must leave the
    device's free memory where it was (nothing allocated behind the caller's back)."""
    M, N, K = 1024, 1024, 4096
    assert q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, q.QNN_ALGO_TC_I8) == q.QNN_NOALLOC_SCRATCH_BYTES
    a, b, ld = _operands(M, N, K, 5)
    got = torch.full((M, N), -9, dtype=torch.int32, device="cuda")
    popc = torch.empty_like(got)
    q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, popc, N, q.QNN_ALGO_POPC)
    q.qnn_xnor_gemm_noalloc(a, ld, b, ld, M, N, K, got, N)        # set-up (first call on this device) happens here at the latest
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        got.fill_(-9)
        q.qnn_xnor_gemm_noalloc(a, ld, b, ld, M, N, K, got, N)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert q.qnn_device_status() == 0
    assert torch.equal(got, popc)


def test_noalloc_rejects_shapes_beyond_the_builtin_scratch(q):
    M = N = K = 4096                              # needs 2 x 16 MiB of int8 operands
    assert q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, q.QNN_ALGO_TC_I8) > q.QNN_NOALLOC_SCRATCH_BYTES
    a, b, ld = _operands(M, N, K, 3)
    out = torch.full((M, N), 5, dtype=torch.int32, device="cuda")
    before = q.qnn_launch_count()
    with pytest.raises(q.QnnError) as e:
        q.qnn_xnor_gemm_noalloc(a, ld, b, ld, M, N, K, out, N)
    assert e.value.status == q.QNN_ERR_WORKSPACE
    assert "built-in" in str(e.value)
    assert q.qnn_launch_count() == before         # nothing was launched
    torch.cuda.synchronize()
    assert bool((out == 5).all())
