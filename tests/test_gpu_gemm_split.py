"""The split-operand projection kernel (two 16-bit planes per fp32 operand, three tensor-core passes, fp32
accumulation) against the plain definition C = A B (+ bias, ReLU, accumulate) computed in fp64 by numpy.
Two fp16 terms carry 22 mantissa bits (two bf16 terms 16), so the result must sit within 1e-4 of the largest
|C| whichever planes are used (a single bf16 pass would be off by 4e-3, one TF32 pass by 1e-3).  K-major products are run on both
forms of the kernel: one CTA per row tile, and pairs of CTAs that share each B tile (one 256-row MMA across two
SMs).  Also: a bounded wait that is made to run out, in either form."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

# (M, N, K, layout): "k" = both operands with the contraction index contiguous (activations [M,K], weights [N,K]);
# "mn" = both with the other index contiguous (C = A^T B, contraction over matrix rows: weight gradients)
SHAPES = [
    (300, 200, 386, "k"),        # key/value projection shape: one pair and a single tile, ragged K (386 = 6*64 + 2)
    (1800, 200, 372, "k"),       # 15 row tiles: 7 pairs and one single
    (5000, 100, 200, "k"),       # 40 row tiles: more work items than a small grid would take at once
    (513, 300, 472, "k"),        # two n-tiles
    (128, 32, 64, "k"),          # one tile, one contraction block
    (5, 7, 3, "k"),              # far below one tile
    (200, 387, 5000, "mn"),      # weight gradient with the bias column: split over the contraction
    (100, 200, 777, "mn"),       # ragged contraction length
    (300, 100, 40, "mn"),        # three row tiles, contraction shorter than two blocks
]


def _operands(rng, M, N, K, lay):
    A = rng.normal(size=(M, K)).astype(np.float32)
    Bm = rng.normal(size=(K, N)).astype(np.float32)
    # values whose low mantissa bits matter: a single bf16 (or tf32) pass would lose them
    A += (rng.integers(0, 2, A.shape) * 2.0 ** -9).astype(np.float32)
    if lay == "k":
        A_dev, sa = torch.from_numpy(A).cuda(), (K, 1)
        B_dev, sb = torch.from_numpy(np.ascontiguousarray(Bm.T)).cuda(), (1, K)     # stored [N, K]
    else:
        A_dev, sa = torch.from_numpy(np.ascontiguousarray(A.T)).cuda(), (1, M)      # stored [K, M]
        B_dev, sb = torch.from_numpy(Bm).cuda(), (N, 1)                             # stored [K, N]
    return A, Bm, A_dev, sa, B_dev, sb


def _scratch(M, N, K):
    up8 = lambda x: (x + 7) // 8 * 8
    n = 4 * (max(M, K) * up8(max(M, K)) + max(N, K) * up8(max(N, K))) + 1024
    return torch.zeros(n, dtype=torch.uint8, device="cuda")


@pytest.fixture(scope="module")
def lib():
    from paper_2608_16305_b200 import binding as B
    l = B.Tgnn(B.make_config(100, 32, 16, 10, 2))
    yield l
    l.close()


PAIR_SHAPES = [
    (300, 200, 386, "k"),        # one 256-row tile and a ragged one whose second half is empty
    (1800, 200, 372, "k"),       # 8 tiles of 256 rows, the last with 8 valid rows
    (513, 300, 472, "k"),        # two n-tiles of different widths; the third tile holds one row
    (40000, 200, 386, "k"),      # 157 tiles over 74 pairs: the persistent walk, accumulators alternating
    (129, 16, 16, "k"),          # narrowest MMA, one contraction step
    (40000, 200, 200, "k"),      # short contraction (the input gradient's shape): tiles of four blocks on a ring of three stages
    (200, 387, 5000, "mn"),      # weight gradient on pairs: two accumulators, 74 parts of the contraction
    (200, 201, 3000, "mn"),      # one accumulator, drained by all eight epilogue warps
    (300, 100, 40, "mn"),        # two 256-row tiles of C, contraction of two blocks
    (256, 512, 777, "mn"),       # the widest C a pair holds; ragged contraction
]


@pytest.mark.parametrize("shape", SHAPES + [s + ("pair",) for s in PAIR_SHAPES])
def test_split_projection_matches_definition(lib, shape, monkeypatch):
    M, N, K, lay = shape[:4]
    monkeypatch.setenv("TGNN_GEMM_PAIR", "1" if len(shape) > 4 else "0")
    rng = np.random.default_rng(M * 1000003 + N * 1009 + K)
    A, Bm, A_dev, sa, B_dev, sb = _operands(rng, M, N, K, lay)
    ref = A.astype(np.float64) @ Bm.astype(np.float64)
    scale = np.abs(ref).max()
    bias = rng.normal(size=N).astype(np.float32)
    scr = _scratch(M, N, K)
    # store mode with bias and ReLU
    C = torch.full((M, N), 7.0, dtype=torch.float32, device="cuda")
    lib.debug_gemm_split(A_dev, *sa, B_dev, *sb, C, N, M, N, K, scr, bias=torch.from_numpy(bias).cuda(), relu=True)
    torch.cuda.synchronize()
    assert lib.status() == 0
    want = np.maximum(ref + bias, 0)
    err = np.abs(C.cpu().numpy() - want).max() / scale
    assert err <= 1e-4, f"store mode err {err}"
    # accumulate mode into a padded C, contraction split over CTAs where it is long enough
    ldc = N + 5
    C0 = rng.normal(size=(M, ldc)).astype(np.float32)
    C = torch.from_numpy(C0.copy()).cuda()
    lib.debug_gemm_split(A_dev, *sa, B_dev, *sb, C, ldc, M, N, K, scr, accumulate=True,
                         split_k=1 if len(shape) > 4 and lay == "k" else 64)   # (K-major pairs do not split the contraction)
    torch.cuda.synchronize()
    assert lib.status() == 0
    got = C.cpu().numpy()
    err = np.abs(got[:, :N] - (C0[:, :N] + ref)).max() / scale
    assert err <= 1e-4, f"accumulate mode err {err}"
    assert np.array_equal(got[:, N:], C0[:, N:])                    # the padding columns are not touched


@pytest.mark.parametrize("shape", [(1800, 200, 372, "k"), (200, 387, 5000, "mn")])
def test_fp16_planes_beat_bf16_planes_and_scaling_keeps_gradients_in_range(lib, shape, monkeypatch):
    """The library holds its operands as two fp16 numbers (22 mantissa bits); the kernel also takes bf16 planes
    (16 bits, any range).  fp16 planes must be the more accurate of the two.  Gradient-sized entries (1e-6) lie
    below fp16's normal range: scaled by 2^12 on the way in (and back in the epilogue) they keep full accuracy."""
    M, N, K, lay = shape
    rng = np.random.default_rng(77)
    A, Bm, A_dev, sa, B_dev, sb = _operands(rng, M, N, K, lay)
    ref = A.astype(np.float64) @ Bm.astype(np.float64)
    scr = _scratch(M, N, K)
    errs = {}
    for bf in ("0", "1"):
        monkeypatch.setenv("TGNN_GEMM_BF16", bf)
        C = torch.zeros((M, N), dtype=torch.float32, device="cuda")
        lib.debug_gemm_split(A_dev, *sa, B_dev, *sb, C, N, M, N, K, scr)
        torch.cuda.synchronize()
        assert lib.status() == 0
        errs[bf] = np.abs(C.cpu().numpy() - ref).max() / np.abs(ref).max()
    # (over a contraction of thousands of terms the fp32 accumulator's own rounding, ~2e-5, hides the difference)
    assert errs["0"] <= 3e-5 and errs["1"] <= 1e-4 and (K > 1000 or errs["0"] < 0.5 * errs["1"]), errs
    monkeypatch.setenv("TGNN_GEMM_BF16", "0")
    small = (A_dev * 1e-6).contiguous()
    for shift, bound in (("0", None), ("12", 5e-6)):
        monkeypatch.setenv("TGNN_GEMM_SCALE", shift)
        C = torch.zeros((M, N), dtype=torch.float32, device="cuda")
        lib.debug_gemm_split(small, *sa, B_dev, *sb, C, N, M, N, K, scr)
        torch.cuda.synchronize()
        errs[shift] = np.abs(C.cpu().numpy() - 1e-6 * ref).max() / np.abs(1e-6 * ref).max()
        if bound:
            assert errs[shift] <= (3e-5 if K > 1000 else bound), errs
    assert errs["12"] < errs["0"], errs          # unscaled, the small entries lose their remainder plane


@pytest.mark.parametrize("shape", [(300, 200, 386, "k"), (1800, 200, 372, "k"), (40000, 200, 386, "k"), (513, 300, 472, "k"),
                                   (200, 387, 5000, "mn"), (100, 200, 777, "mn"), (256, 512, 777, "mn")])
def test_single_pass_products_hold_fp16_accuracy(lib, shape, monkeypatch):
    """Only the hi plane of each operand and one tensor-core pass: the form the step uses for the key/value weight
    gradient when the feature table is bf16 (tolerance 1e-2).  Eleven
    mantissa bits per operand: the product of random operands stays within 1e-3 of the largest |C| (three passes:
    1e-4), through every kernel form the launcher picks for the shape."""
    M, N, K, lay = shape
    monkeypatch.setenv("TGNN_GEMM_PASSES", "1")
    monkeypatch.delenv("TGNN_GEMM_PAIR", raising=False)
    rng = np.random.default_rng(M + 7 * N + 13 * K)
    A, Bm, A_dev, sa, B_dev, sb = _operands(rng, M, N, K, lay)
    ref = A.astype(np.float64) @ Bm.astype(np.float64)
    scr = _scratch(M, N, K)
    bias = rng.normal(size=N).astype(np.float32)
    C = torch.full((M, N), 7.0, dtype=torch.float32, device="cuda")
    lib.debug_gemm_split(A_dev, *sa, B_dev, *sb, C, N, M, N, K, scr, bias=torch.from_numpy(bias).cuda())
    torch.cuda.synchronize()
    assert lib.status() == 0
    err = np.abs(C.cpu().numpy() - (ref + bias)).max() / np.abs(ref).max()
    assert 1e-6 < err <= 1e-3, err          # (far above the three-pass error: the lo planes really are not used)
    ldc = (N + 3) // 4 * 4
    C0 = rng.normal(size=(M, ldc)).astype(np.float32)
    C = torch.from_numpy(C0.copy()).cuda()
    lib.debug_gemm_split(A_dev, *sa, B_dev, *sb, C, ldc, M, N, K, scr, accumulate=True, split_k=64 if lay == "mn" else 1)
    torch.cuda.synchronize()
    assert lib.status() == 0
    err = np.abs(C.cpu().numpy()[:, :N] - (C0[:, :N] + ref)).max() / np.abs(ref).max()
    assert err <= 1e-3, err


def test_every_tile_lands_where_the_definition_puts_it(lib):
    """Index-valued operands: A picks row m of B scaled by a small integer, so every C entry names the (row
    tile, n-tile, column) it came from exactly (all values are small integers, exact in bf16)."""
    M, N, K = 700, 300, 192
    A = np.zeros((M, K), np.float32)
    A[np.arange(M), np.arange(M) % K] = 1.0 + (np.arange(M) // K)
    Bm = (np.arange(K)[:, None] * 2 + (np.arange(N)[None, :] % 2)).astype(np.float32)      # < 512: exact in bf16
    want = A.astype(np.float64) @ Bm.astype(np.float64)
    scr = _scratch(M, N, K)
    for lay in ("k", "mn"):
        if lay == "k":
            A_dev, sa, B_dev, sb = torch.from_numpy(A).cuda(), (K, 1), torch.from_numpy(np.ascontiguousarray(Bm.T)).cuda(), (1, K)
        else:
            A_dev, sa, B_dev, sb = torch.from_numpy(np.ascontiguousarray(A.T)).cuda(), (1, M), torch.from_numpy(Bm).cuda(), (N, 1)
        C = torch.full((M, N), -1.0, dtype=torch.float32, device="cuda")
        lib.debug_gemm_split(A_dev, *sa, B_dev, *sb, C, N, M, N, K, scr)
        torch.cuda.synchronize()
        assert lib.status() == 0
        assert np.array_equal(C.cpu().numpy(), want), lay


@pytest.mark.parametrize("pair", [0, 1])
def test_a_wait_that_runs_out_is_reported_and_leaves_the_context_usable(lib, pair, monkeypatch):
    """The kernel's waits are bounded.  With one shared-memory slot withheld (a debug hook: the MMA warp does
    not hand it back) and a short limit, the copy warp's wait for that slot runs out: the kernel records
    TGNN_ETIMEOUT in the status word, stores nothing, frees its tensor memory and returns.  A normal launch
    right after it (which needs that tensor memory) gives the right answer.  In the paired form both CTAs' copy
    warps run out, each raises the other's abort flag, and the two meet at the cluster barrier before they free
    tensor memory."""
    from paper_2608_16305_b200 import binding as B
    monkeypatch.setenv("TGNN_GEMM_PAIR", str(pair))
    M, N, K = 128 * (1 + pair), 64, 4096          # one work item, 64 contraction blocks: more than the ring holds
    rng = np.random.default_rng(5)
    A, Bm, A_dev, sa, B_dev, sb = _operands(rng, M, N, K, "k")
    scr = _scratch(M, N, K)
    C = torch.full((M, N), 3.0, dtype=torch.float32, device="cuda")
    lib.debug_gemm_split(A_dev, *sa, B_dev, *sb, C, N, M, N, K, scr, debug_withhold=1, spin_limit=1 << 12)
    torch.cuda.synchronize()
    assert lib.status() == B.TGNN_ETIMEOUT
    assert bool((C == 3.0).all())                 # the epilogue never ran
    lib.clear_status()
    lib.debug_gemm_split(A_dev, *sa, B_dev, *sb, C, N, M, N, K, scr)
    torch.cuda.synchronize()
    assert lib.status() == 0
    ref = A.astype(np.float64) @ Bm.astype(np.float64)
    assert np.abs(C.cpu().numpy() - ref).max() / np.abs(ref).max() <= 1e-4
