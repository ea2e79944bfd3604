"""The dense-projection kernels against the plain definition C = A B (+ bias, ReLU, accumulate),
computed in fp64 by numpy: fp32 FMA tiles to 1e-5 of the largest |C|, the 3xTF32 head/tail split to 1e-4 (contractions up to 5000),
plain TF32 tensor-core tiles to 2e-3 (operands rounded to 10 mantissa bits)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

# (M, N, K, A layout, B layout): layouts name which index is contiguous in memory
SHAPES = [
    (300, 100, 200, "k", "k"),      # forward projection: activations [M,K] x weights [N,K]
    (1800, 200, 372, "k", "k"),     # key/value projection (ragged K: 372 = 11*32 + 20, N = 200)
    (513, 300, 472, "k", "k"),      # GRU input gates: two n-tiles
    (1000, 100, 200, "k", "mn"),    # input gradient: dY [M,N'] x W [N',K]
    (200, 372, 5000, "mn", "mn"),   # weight gradient: dY^T x Z, contraction over rows, split-K
    (100, 200, 777, "mn", "mn"),    # small weight gradient, ragged contraction
    (128, 32, 32, "k", "k"),        # a single stage
    (5, 7, 3, "k", "k"),            # far below one tile, unaligned everything
    (260, 200, 386, "k", "k"),      # row stride 386 floats: rows not 16-byte aligned
]


def _operands(rng, M, N, K, la, lb, pad=0):
    A = rng.normal(size=(M, K)).astype(np.float32)
    Bm = rng.normal(size=(K, N)).astype(np.float32)
    if la == "k":
        A_dev = torch.from_numpy(np.ascontiguousarray(np.pad(A, ((0, 0), (0, pad))))).cuda()
        a_rs, a_cs = K + pad, 1
    else:
        A_dev = torch.from_numpy(np.ascontiguousarray(np.pad(A.T, ((0, 0), (0, pad))))).cuda()     # stored [K, M]
        a_rs, a_cs = 1, M + pad
    if lb == "k":
        B_dev = torch.from_numpy(np.ascontiguousarray(np.pad(Bm.T, ((0, 0), (0, pad))))).cuda()    # stored [N, K]
        b_rs, b_cs = 1, K + pad
    else:
        B_dev = torch.from_numpy(np.ascontiguousarray(np.pad(Bm, ((0, 0), (0, pad))))).cuda()      # stored [K, N]
        b_rs, b_cs = N + pad, 1
    return A, Bm, A_dev, (a_rs, a_cs), B_dev, (b_rs, b_cs)


@pytest.mark.parametrize("mode", ["fp32", "tf32", "tf32x3"])
@pytest.mark.parametrize("shape", SHAPES)
def test_projection_matches_definition(mode, shape):
    from paper_2608_16305_b200 import binding as B
    M, N, K, la, lb = shape
    rng = np.random.default_rng(M * 1000003 + N * 1009 + K)
    lib = B.Tgnn(B.make_config(100, 32, 16, 10, 2, math_mode=B.TGNN_MATH_FP32 if mode == "fp32" else B.TGNN_MATH_TF32_FAST))
    tol = {"fp32": 1e-5, "tf32": 2e-3, "tf32x3": 1e-4}[mode]
    precise = mode == "tf32x3"
    A, Bm, A_dev, sa, B_dev, sb = _operands(rng, M, N, K, la, lb)
    ref = A.astype(np.float64) @ Bm.astype(np.float64)
    bias = rng.normal(size=N).astype(np.float32)
    scale = np.abs(ref).max()
    # store mode with bias and ReLU
    C = torch.full((M, N), 7.0, dtype=torch.float32, device="cuda")
    lib.debug_gemm(A_dev, *sa, B_dev, *sb, C, N, M, N, K, bias=torch.from_numpy(bias).cuda(), relu=True, precise=precise)
    torch.cuda.synchronize()
    assert lib.status() == 0
    want = np.maximum(ref + bias, 0)
    assert np.abs(C.cpu().numpy() - want).max() <= tol * scale
    # accumulate mode with split-K and the row sums of A (only transposed products use them)
    C0 = rng.normal(size=(M, N)).astype(np.float32)
    C = torch.from_numpy(C0.copy()).cuda()
    rs = torch.zeros(M, dtype=torch.float32, device="cuda") if la == "mn" else None
    lib.debug_gemm(A_dev, *sa, B_dev, *sb, C, N, M, N, K, rowsum_out=rs, accumulate=True, split_k=8, precise=precise)
    torch.cuda.synchronize()
    assert lib.status() == 0
    assert np.abs(C.cpu().numpy() - (ref + C0)).max() <= tol * scale
    if rs is not None:
        want_rs = A.astype(np.float64).sum(1)
        assert np.abs(rs.cpu().numpy() - want_rs).max() <= 1e-4 * max(np.abs(A).sum(1).max(), 1.0)
    # device-side counts smaller than the capacities
    if M > 8 and K > 40:
        m_dev = torch.tensor([M - 5], dtype=torch.int32, device="cuda")
        k_dev = torch.tensor([K - 37], dtype=torch.int32, device="cuda")
        C = torch.full((M, N), 7.0, dtype=torch.float32, device="cuda")
        lib.debug_gemm(A_dev, *sa, B_dev, *sb, C, N, M, N, K, dev_M=m_dev if la == "k" else None,
                       dev_K=k_dev if la == "mn" else None, precise=precise)
        torch.cuda.synchronize()
        got = C.cpu().numpy()
        if la == "k":
            assert np.abs(got[:M - 5] - ref[:M - 5]).max() <= tol * scale and (got[M - 5:] == 7.0).all()
        else:
            ref2 = A[:, :K - 37].astype(np.float64) @ Bm[:K - 37].astype(np.float64)
            assert np.abs(got - ref2).max() <= tol * scale
    lib.close()


@pytest.mark.parametrize("M,N,K,pad", [
    (192, 352, 4096, 0),     # widths are whole 32-column atoms
    (200, 372, 5000, 28),    # ragged widths inside padded rows: the last atom of a row reads the padding
    (100, 200, 1200, 24),    # one tile, split-K, several contraction blocks per CTA
    (128, 256, 36, 0),       # contraction shorter than two blocks, a full 256-column tile
])
def test_transposed_products_by_tiles(M, N, K, pad):
    """Weight-gradient shaped products (both operands transposed, contraction over rows) whose operands are
    delivered by the tensor-memory-access unit: widths that are whole atoms, or rows padded far enough that the
    last atom stays inside the matrix (the library does not read past a caller's buffer)."""
    from paper_2608_16305_b200 import binding as B
    rng = np.random.default_rng(M + 7 * N + 13 * K)
    lib = B.Tgnn(B.make_config(100, 32, 16, 10, 2, math_mode=B.TGNN_MATH_TF32))
    A, Bm, A_dev, sa, B_dev, sb = _operands(rng, M, N, K, "mn", "mn", pad=pad)
    ref = A.astype(np.float64) @ Bm.astype(np.float64)
    scale = np.abs(ref).max()
    C0 = rng.normal(size=(M, N)).astype(np.float32)
    for split in (1, 8):
        C = torch.from_numpy(C0.copy()).cuda()
        rs = torch.zeros(M, dtype=torch.float32, device="cuda")
        lib.debug_gemm(A_dev, *sa, B_dev, *sb, C, N, M, N, K, rowsum_out=rs, accumulate=True, split_k=split, precise=True)
        torch.cuda.synchronize()
        assert lib.status() == 0
        assert np.abs(C.cpu().numpy() - (ref + C0)).max() <= 1e-4 * scale
        assert np.abs(rs.cpu().numpy() - A.astype(np.float64).sum(1)).max() <= 1e-4 * max(np.abs(A).sum(1).max(), 1.0)
    lib.close()


@pytest.mark.parametrize("layout", [("mn", "mn"), ("k", "k"), ("k", "mn")])
@pytest.mark.parametrize("low_bits", [0x1fff, 0x1000, 0x0fff])
def test_operand_split_keeps_the_low_mantissa_bits(layout, low_bits):
    """Positive operands whose 13 low mantissa bits are all set (or exactly half / just under half an ulp of
    the 10-bit head): any mismatch between how the head is formed and what the tensor core takes as the head
    -- rounding on one side, truncation on the other -- shifts every product by up to 2^-10 in the same
    direction, a relative error near 1e-3 on these all-positive sums.  The split product must stay near the
    fp32 level instead (the bound leaves room for the accumulator's own rounding over the 96 accumulation
    steps of K = 256, which on all-positive sums adds up to a few 1e-6)."""
    from paper_2608_16305_b200 import binding as B
    M, N, K = 128, 160, 256
    rng = np.random.default_rng(low_bits)
    lib = B.Tgnn(B.make_config(100, 32, 16, 10, 2, math_mode=B.TGNN_MATH_TF32))

    def worst(shape):
        x = (1.0 + rng.random(shape)).astype(np.float32)
        return ((x.view(np.uint32) & np.uint32(0xffffe000)) | np.uint32(low_bits)).view(np.float32)
    A, Bm = worst((M, K)), worst((K, N))
    la, lb = layout
    if la == "k":
        A_dev, sa = torch.from_numpy(A).cuda(), (K, 1)
    else:
        A_dev, sa = torch.from_numpy(np.ascontiguousarray(A.T)).cuda(), (1, M)
    if lb == "k":
        B_dev, sb = torch.from_numpy(np.ascontiguousarray(Bm.T)).cuda(), (1, K)
    else:
        B_dev, sb = torch.from_numpy(Bm).cuda(), (N, 1)
    ref = A.astype(np.float64) @ Bm.astype(np.float64)
    for acc, split in ((False, 1), (True, 4)):
        C = torch.zeros((M, N), dtype=torch.float32, device="cuda")
        lib.debug_gemm(A_dev, *sa, B_dev, *sb, C, N, M, N, K, accumulate=acc, split_k=split, precise=True)
        torch.cuda.synchronize()
        assert lib.status() == 0
        err = np.abs(C.cpu().numpy() - ref).max() / ref.max()
        assert err <= 2e-5, (layout, hex(low_bits), acc, err)
    lib.close()
