"""Parity of the FP16 GEMMs (FP32 accumulate, FP16 store; paper section 3.3) with the oracle.

The CUDA-core kernel sums in the oracle's order and must match bit for bit; the
tensor-core kernel sums in hardware order and is held to the acceptance rule
(2 FP16 ulp / 1e-2 relative / a-priori summation bound near zero)."""
import numpy as np
import pytest

from oracle import mpo
from paper_1710_03740_b200 import inputs
from parity import gemm_accept
from gpu_util import dev, host_u16, require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def _pad(a, ld):
    rows, cols = a.shape
    out = np.zeros((rows, ld), dtype=np.uint16)
    out[:, :cols] = a.view(np.uint16)
    return out


def run_gemm(op, A, B, M, N, K, flags=0, mask=None, pad=0, want_flag=False, workspace=False):
    """A, B: stored float16 operands.  pad: extra columns added to every pitch."""
    from paper_1710_03740_b200 import binding as b
    lda, ldb, ldc = A.shape[1] + pad, B.shape[1] + pad, N + pad
    Ad, Bd = dev(_pad(A, lda)), dev(_pad(B, ldb))
    Cd = torch.full((M, ldc), 0x5555, dtype=torch.int16, device="cuda")
    md = dev(_pad(mask, ldc)) if mask is not None else None
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    if workspace:
        nbytes = b.mpt_gemm_workspace_bytes(op, M, N, K)
        if nbytes == 0 and not flags & (b.GEMM_FORCE_TC | b.GEMM_FORCE_PAIR):
            pytest.skip("the library's own choice needs no scratch for this shape")
        # room for any split either kernel may choose (the need reported is that of the automatic choice)
        nbytes = max(nbytes, 9 * M * ((N + 31) // 32 * 32) * 4)
        ws = torch.full((nbytes // 4,), float("nan"), dtype=torch.float32, device="cuda")
        b.mpt_gemm_f16_ws(op, M, N, K, Ad, lda, Bd, ldb, Cd, ldc, flags, md, ldc if mask is not None else 0,
                          flag if want_flag else None, status, ws)
    else:
        b.mpt_gemm_f16(op, M, N, K, Ad, lda, Bd, ldb, Cd, ldc, flags, md, ldc if mask is not None else 0,
                       flag if want_flag else None, status)
    torch.cuda.synchronize()
    assert int(status[0].item()) == 0, "device-side wait expired: 0x%x" % int(status[0].item())
    out = host_u16(Cd)
    if pad:
        assert np.all(out[:, N:] == 0x5555)
    return out[:, :N], int(flag.item())


SIMT_SHAPES = [(1, 1, 1), (5, 7, 3), (64, 10, 512), (70, 130, 33), (129, 65, 100), (256, 256, 64)]


@pytest.mark.parametrize("op", [0, 1, 2])
@pytest.mark.parametrize("M,N,K", SIMT_SHAPES)
def test_simt_gemm_bit_exact(op, M, N, K):
    from paper_1710_03740_b200 import binding as b
    A, B = inputs.gemm_operands(op, M, N, K, seed=11, scale_a=1.0, scale_b=1.0)
    ref = mpo.gemm_f16(op, A, B)
    got, _ = run_gemm(op, A, B, M, N, K, flags=b.GEMM_FORCE_SIMT, pad=3)
    assert np.array_equal(got, ref)


def test_simt_gemm_relu_mask_flag():
    from paper_1710_03740_b200 import binding as b
    M, N, K = 50, 40, 64
    A, B = inputs.gemm_operands(0, M, N, K, seed=12, scale_a=1.0, scale_b=1.0)
    ref = mpo.gemm_f16(0, A, B, relu=True)
    got, _ = run_gemm(0, A, B, M, N, K, flags=b.GEMM_FORCE_SIMT | b.GEMM_RELU)
    assert np.array_equal(got, ref)
    rng = np.random.default_rng(1)
    mask = rng.standard_normal((M, N)).astype(np.float16)
    mask[0, :4] = [0.0, -0.0, np.nan, np.inf]
    A, B = inputs.gemm_operands(1, M, N, K, seed=13, scale_a=1.0, scale_b=1.0)
    ref = mpo.gemm_f16(1, A, B, mask=mask)
    got, flag = run_gemm(1, A, B, M, N, K, flags=b.GEMM_FORCE_SIMT, mask=mask, want_flag=True)
    assert np.array_equal(got, ref) and flag == 0
    A2 = (A.astype(np.float32) * 3000).astype(np.float16)
    B2 = (B.astype(np.float32) * 3000).astype(np.float16)
    ref = mpo.gemm_f16(1, A2, B2)
    got, flag = run_gemm(1, A2, B2, M, N, K, flags=b.GEMM_FORCE_SIMT, want_flag=True)
    assert np.array_equal(got, ref)
    assert flag == 1 and (~np.isfinite(ref.view(np.float16).astype(np.float32))).any()


_ORACLE_CACHE = {}


def _check_tc(op, M, N, K, flags=0, mask=None, seed=21, scale=None, want_flag=False, kernel="tc", workspace=False):
    from paper_1710_03740_b200 import binding as b
    force = {"pair": b.GEMM_FORCE_PAIR, "tc": b.GEMM_FORCE_TC, "auto": 0, "pair512": b.GEMM_FORCE_PAIR512,
             "split2": b.GEMM_FORCE_SPLIT2, "split4": b.GEMM_FORCE_SPLIT4}[kernel]
    sa = sb = scale
    key = (op, M, N, K, seed, scale, bool(flags & b.GEMM_RELU))
    if mask is None and key in _ORACLE_CACHE:        # the oracle is slow: keep its answer for repeated inputs
        A, B, ref, ex, ab = _ORACLE_CACHE[key]
    else:
        A, B = inputs.gemm_operands(op, M, N, K, seed=seed, scale_a=sa, scale_b=sb)
        ref, ex, ab = mpo.gemm_f16(op, A, B, relu=bool(flags & b.GEMM_RELU), mask=mask, want_exact=True)
        if mask is None:
            if len(_ORACLE_CACHE) >= 4:
                _ORACLE_CACHE.pop(next(iter(_ORACLE_CACHE)))
            _ORACLE_CACHE[key] = (A, B, ref, ex, ab)
    got, flag = run_gemm(op, A, B, M, N, K, flags=flags | force, mask=mask,
                         pad=(8 if (M * N) % 3 == 0 else 0), want_flag=want_flag, workspace=workspace)
    ok, stats = gemm_accept(got, ref, K=K, absdot=ab, exact=ex)
    assert ok.all(), (op, M, N, K, stats, np.argwhere(~ok)[:8].tolist())
    assert stats["by_abs_only"] <= max(2, stats["n"] // 1000), stats
    # both sides within the summation bound of the exactly rounded sum
    if not flags and mask is None:
        with np.errstate(over="ignore"):      # sums beyond the FP16 range become inf, as intended
            exact16 = ex.astype(np.float32).astype(np.float16).view(np.uint16)
        ok2, st2 = gemm_accept(got, exact16, K=K, absdot=ab, exact=ex)
        assert ok2.all(), st2
    return got, ref, flag, stats


TC_SHAPES = [(128, 256, 64), (128, 256, 256), (256, 512, 128), (128, 256, 72), (200, 304, 136),
             (64, 16, 512), (8, 8, 8), (384, 768, 1024), (1024, 1024, 1024),
             (1000, 1016, 1032)]      # the last two take 128x64 tiles (ragged in every dimension here)


PAIR_SHAPES = [(256, 256, 64), (256, 256, 448), (512, 768, 128), (256, 512, 72), (392, 560, 136),
                (64, 16, 512), (8, 8, 8), (1280, 1024, 1024)]


@pytest.mark.parametrize("op", [0, 1, 2])
@pytest.mark.parametrize("M,N,K", TC_SHAPES)
def test_tc_gemm_parity(op, M, N, K):
    _check_tc(op, M, N, K)


@pytest.mark.parametrize("op", [0, 1, 2])
@pytest.mark.parametrize("M,N,K", PAIR_SHAPES)
def test_pair_gemm_parity(op, M, N, K):
    _check_tc(op, M, N, K, kernel="pair")


@pytest.mark.parametrize("op", [0, 1, 2])
def test_sweep_2048_cubed_in_full_every_kernel(op):
    """2048^3 of the isolated-GEMM sweep (seed and operand distribution of that sweep), every
    output element against the oracle: under the library's own kernel choice with and without a
    scratch buffer, and with each tensor-core kernel forced.  The automatic choice changes hands
    near this size (64 tiles of 256x256: the last shape of the sweep the single-CTA kernel takes)."""
    from paper_1710_03740_b200 import binding as b
    M = N = K = 2048
    assert (M, N, K) in inputs.GEMM_SWEEP
    auto, _, _, _ = _check_tc(op, M, N, K, seed=2, kernel="auto")
    again, _, _, _ = _check_tc(op, M, N, K, seed=2, kernel="auto")
    assert np.array_equal(auto, again)
    for kernel in ("tc", "pair", "pair512"):
        _check_tc(op, M, N, K, seed=2, kernel=kernel)
    if b.mpt_gemm_workspace_bytes(op, M, N, K):
        _check_tc(op, M, N, K, seed=2, kernel="auto", workspace=True)


PAIR512_SHAPES = [(256, 512, 64), (256, 512, 448), (512, 1536, 128), (256, 768, 72), (392, 1080, 136), (264, 264, 200),
                  (64, 16, 512), (8, 8, 8), (1280, 2048, 1024), (256, 256, 320)]


@pytest.mark.parametrize("op", [0, 1, 2])
@pytest.mark.parametrize("M,N,K", PAIR512_SHAPES)
def test_pair512_gemm_parity(op, M, N, K):
    """CTA-pair kernel with 256x512 tiles: whole tiles, ragged right edges wider and narrower than
    one accumulator, ragged M and K, and shapes smaller than a tile."""
    _check_tc(op, M, N, K, kernel="pair512")


@pytest.mark.parametrize("op", [0, 1, 2])
def test_pair512_many_tiles_halves_relu_mask_flag(op):
    """More tiles than clusters (the ring, the accumulator hand-over and the K direction all
    alternate several times), a last round cut into 256-column halves, ReLU / mask / overflow flag
    through the two epilogue sets, and identical bits on a rerun."""
    from paper_1710_03740_b200 import binding as b
    M, N, K = 2304, 5120 + 256, 136            # 9 x 11 tiles: 74 whole tiles, 25 cut into halves
    got, _, _, _ = _check_tc(op, M, N, K, kernel="pair512")
    again, _, _, _ = _check_tc(op, M, N, K, kernel="pair512")
    assert np.array_equal(got, again)
    M, N, K = 512, 1024, 320
    _check_tc(op, M, N, K, flags=b.GEMM_RELU, kernel="pair512")
    mask = np.random.default_rng(9).standard_normal((M, N)).astype(np.float16)
    _check_tc(op, M, N, K, mask=mask, kernel="pair512")
    _, ref, flag, _ = _check_tc(op, M, N, K, scale=40.0, want_flag=True, kernel="pair512")
    assert flag == int(((ref & 0x7FFF) >= 0x7C00).any()) == 1
    _, _, flag, _ = _check_tc(op, M, N, K, want_flag=True, kernel="pair512")
    assert flag == 0


CLUSTER_SPLIT_SHAPES = [(256, 256, 256), (256, 256, 448), (512, 768, 1024), (392, 560, 328), (264, 264, 2056),
                        (64, 16, 512), (8, 8, 256), (1024, 1024, 4096)]


@pytest.mark.parametrize("kernel", ["split2", "split4"])
@pytest.mark.parametrize("op", [0, 1, 2])
@pytest.mark.parametrize("M,N,K", CLUSTER_SPLIT_SHAPES)
def test_cluster_split_gemm_parity(op, M, N, K, kernel):
    """In-cluster split of the contraction (2 or 4 CTA pairs per tile, parts added through distributed
    shared memory): one tile and several, parts of unequal length (7, 6, 33 k-blocks), ragged M, N and
    K, shapes smaller than a tile, and more clusters than the GPU holds at once (16 tiles of 8 CTAs)."""
    _check_tc(op, M, N, K, kernel=kernel)


@pytest.mark.parametrize("kernel", ["split2", "split4"])
@pytest.mark.parametrize("op", [0, 1, 2])
def test_cluster_split_relu_mask_flag_and_rerun(op, kernel):
    from paper_1710_03740_b200 import binding as b
    M, N, K = 520, 776, 1352
    got, _, _, _ = _check_tc(op, M, N, K, kernel=kernel)
    again, _, _, _ = _check_tc(op, M, N, K, kernel=kernel)
    assert np.array_equal(got, again)
    _check_tc(op, M, N, K, flags=b.GEMM_RELU, kernel=kernel)
    mask = np.random.default_rng(10).standard_normal((M, N)).astype(np.float16)
    _check_tc(op, M, N, K, mask=mask, kernel=kernel)
    _, ref, flag, _ = _check_tc(op, M, N, K, scale=30.0, want_flag=True, kernel=kernel)
    assert flag == int(((ref & 0x7FFF) >= 0x7C00).any()) == 1
    _, _, flag, _ = _check_tc(op, M, N, K, want_flag=True, kernel=kernel)
    assert flag == 0


def test_cluster_split_is_the_automatic_choice_for_the_projection_shape():
    """Section 4.5's projection product (2048 x 1024 x 8192: 32 tiles, 128 k-blocks): the library picks
    the in-cluster split by itself, needs no scratch for it, and gives the bits of the forced kernel."""
    from paper_1710_03740_b200 import binding as b
    M, N, K = 2048, 1024, 8192
    assert b.mpt_gemm_workspace_bytes(0, M, N, K) == 0
    auto, _, _, _ = _check_tc(0, M, N, K, seed=5, kernel="auto")
    forced, _, _, _ = _check_tc(0, M, N, K, seed=5, kernel="split2")
    assert np.array_equal(auto, forced)
    with pytest.raises(b.MptError):          # a part must have at least one k-block
        _check_tc(0, 256, 256, 64, kernel="split2")


@pytest.mark.parametrize("M,N,K,same_as", [(1024, 768, 4096, "split4"), (1024, 1024, 4096, "split2"),
                                            (512, 512, 2048, "split2"), (512, 512, 1984, "tc"), (2048, 1280, 2048, "tc")])
def test_automatic_kernel_choice_around_the_split_thresholds(M, N, K, same_as):
    """Which kernel the library picks by itself, shown by the bits: 12 tiles with K = 4096 take four
    parts, 16 tiles two parts, 4 tiles with 32 k-blocks two parts, one k-block fewer or 40 tiles none
    (single-CTA kernel) - each result equal to that kernel forced, and all within the acceptance rule."""
    from paper_1710_03740_b200 import binding as b
    assert b.mpt_gemm_workspace_bytes(0, M, N, K) == 0 or same_as == "tc"
    auto, _, _, _ = _check_tc(0, M, N, K, seed=7, kernel="auto")
    forced, _, _, _ = _check_tc(0, M, N, K, seed=7, kernel=same_as)
    assert np.array_equal(auto, forced)
    if same_as != "tc":
        other, _, _, _ = _check_tc(0, M, N, K, seed=7, kernel="tc")
        assert not np.array_equal(auto, other)          # a split sum rounds differently somewhere


def _random_shapes(n, seed):
    """Seeded shapes with every dimension a multiple of 8 (what the tensor-core kernels take), spread over
    the regions of the kernel choice: few tiles with a long contraction (in-cluster split), up to 74 tiles
    (single-CTA kernel), more (CTA pair, with and without a ragged last round), and narrow outputs."""
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        kind = len(out) % 4
        if kind == 0:      # few tiles, long K
            M, N, K = 8 * rng.integers(32, 96), 8 * rng.integers(32, 96), 8 * rng.integers(256, 640)
        elif kind == 1:    # mid-size
            M, N, K = 8 * rng.integers(64, 260), 8 * rng.integers(64, 260), 8 * rng.integers(8, 96)
        elif kind == 2:    # many tiles, short K
            M, N, K = 8 * rng.integers(260, 420), 8 * rng.integers(260, 420), 8 * rng.integers(4, 24)
        else:              # thin
            M, N, K = 8 * rng.integers(1, 24), 8 * rng.integers(1, 200), 8 * rng.integers(8, 400)
        if M * N * K <= 1.6e9:
            out.append((int(M), int(N), int(K)))
    return out


@pytest.mark.parametrize("idx", range(24))
def test_random_shapes_under_the_automatic_choice(idx):
    """The library's own kernel choice on seeded random shapes, one of the three product forms each, with a
    scratch buffer where the choice wants one, plus ReLU on every third: every element within the
    acceptance rule against the oracle."""
    from paper_1710_03740_b200 import binding as b
    M, N, K = _random_shapes(24, 2024)[idx]
    op = idx % 3
    flags = b.GEMM_RELU if idx % 3 == 0 else 0
    ws = b.mpt_gemm_workspace_bytes(op, M, N, K) > 0
    _check_tc(op, M, N, K, flags=flags, seed=100 + idx, kernel="auto", workspace=ws)


@pytest.mark.parametrize("kernel", ["tc", "pair"])
@pytest.mark.parametrize("op", [0, 1, 2])
def test_tc_gemm_run_to_run_identical(op, kernel):
    M, N, K = 304, 520, 392
    a, _, _, _ = _check_tc(op, M, N, K, kernel=kernel)
    b2, _, _, _ = _check_tc(op, M, N, K, kernel=kernel)
    assert np.array_equal(a, b2)


def test_pair_kernel_runs_many_tiles_per_cluster():
    """More 256x256 tiles than clusters: the ring, the two accumulator buffers and the
    barrier phases all wrap several times."""
    _check_tc(0, 2048, 4096 + 256, 192, kernel="pair")
    _check_tc(2, 2304, 3072, 136, kernel="pair")


@pytest.mark.parametrize("op", [0, 1, 2])
def test_pair_kernel_tensor_store_epilogue(op):
    """Long main loops take the epilogue that stages 32 x 64 boxes in shared memory and writes them with
    tensor stores: ragged M and N (boxes cut by the matrix edge, boxes wholly outside), ReLU, the ReLU mask,
    the overflow flag, identical bits on a rerun and identical bits to the per-lane stores."""
    import os
    from paper_1710_03740_b200 import binding as b
    M, N, K = 520, 776, 10304            # 161 k-blocks: one epilogue warp set; 3 x 4 tiles, the last ones ragged
    got, _, _, _ = _check_tc(op, M, N, K, kernel="pair")
    again, _, _, _ = _check_tc(op, M, N, K, kernel="pair")
    assert np.array_equal(got, again)
    os.environ["MPT_TMA_STORE"] = "0"
    try:
        plain, _, _, _ = _check_tc(op, M, N, K, kernel="pair")
    finally:
        del os.environ["MPT_TMA_STORE"]
    assert np.array_equal(got, plain)
    _check_tc(op, M, N, K, flags=b.GEMM_RELU, kernel="pair")
    mask = np.random.default_rng(11).standard_normal((M, N)).astype(np.float16)
    _check_tc(op, M, N, K, mask=mask, kernel="pair")
    _, ref, flag, _ = _check_tc(op, M, N, K, scale=30.0, want_flag=True, kernel="pair")
    assert flag == int(((ref & 0x7FFF) >= 0x7C00).any()) == 1
    _, _, flag, _ = _check_tc(op, M, N, K, want_flag=True, kernel="pair")
    assert flag == 0


@pytest.mark.parametrize("op", [0, 1, 2])
@pytest.mark.parametrize("M,N,K", [(1280, 4000, 136), (1280, 3944, 72), (2304, 3072, 200)])
def test_pair_kernel_half_width_tail_units(op, M, N, K):
    """A few more tiles than clusters: the left-over tiles run as two 256x128 halves, including
    halves that are partly or wholly outside a ragged N."""
    _check_tc(op, M, N, K, kernel="pair")


@pytest.mark.parametrize("op", [0, 1, 2])
@pytest.mark.parametrize("M,N,K", [(512, 256, 4096), (256, 264, 8192), (136, 96, 8192), (384, 1024, 6144)])
def test_split_k_parity_and_determinism(op, M, N, K):
    """Few output tiles and a long contraction: the contraction is split over CTAs, FP32 parts are
    added in a fixed order by a second kernel.  Same acceptance rule; identical bits on a rerun;
    ReLU, mask and the overflow flag go through the reduce kernel."""
    from paper_1710_03740_b200 import binding as b
    if (M, N, K) == (136, 96, 8192):
        assert b.mpt_gemm_workspace_bytes(op, M, N, K) > 0      # few tiles, long K, too small for a CTA pair: must split
    got, ref, _, _ = _check_tc(op, M, N, K, workspace=True)
    again, _, _, _ = _check_tc(op, M, N, K, workspace=True)
    assert np.array_equal(got, again)
    _check_tc(op, M, N, K, flags=b.GEMM_RELU, workspace=True)
    mask = np.random.default_rng(8).standard_normal((M, N)).astype(np.float16)
    _check_tc(op, M, N, K, mask=mask, workspace=True)
    _, ref, flag, _ = _check_tc(op, M, N, K, scale=30.0, want_flag=True, workspace=True)
    assert flag == int(((ref & 0x7FFF) >= 0x7C00).any()) == 1


@pytest.mark.parametrize("op", [0, 1, 2])
@pytest.mark.parametrize("M,N,K", [(512, 512, 4096), (1024, 512, 8192), (264, 520, 2056), (2048, 1024, 8192)])
def test_pair_kernel_split_k(op, M, N, K):
    """Few 256x256 tiles and a long contraction on the CTA-pair kernel: the contraction is split over
    clusters and the FP32 parts are added in ascending order by the reduce kernel.  Same acceptance
    rule; identical bits on reruns; ReLU, mask and the overflow flag go through the reduce kernel; a
    scratch full of NaN bits is fine."""
    from paper_1710_03740_b200 import binding as b
    big = (M, N, K) == (2048, 1024, 8192)
    got, ref, _, _ = _check_tc(op, M, N, K, workspace=True, kernel="pair")
    for _ in range(3):
        again, _, _, _ = _check_tc(op, M, N, K, workspace=True, kernel="pair")
        assert np.array_equal(got, again)
    _check_tc(op, M, N, K, kernel="auto")        # the library's own choice here is the in-cluster split: no scratch
    if not big:
        _check_tc(op, M, N, K, flags=b.GEMM_RELU, workspace=True, kernel="pair")
        mask = np.random.default_rng(8).standard_normal((M, N)).astype(np.float16)
        _check_tc(op, M, N, K, mask=mask, workspace=True, kernel="pair")
        _, ref, flag, _ = _check_tc(op, M, N, K, scale=30.0, want_flag=True, workspace=True, kernel="pair")
        assert flag == int(((ref & 0x7FFF) >= 0x7C00).any()) == 1


@pytest.mark.parametrize("op", [0, 1, 2])
@pytest.mark.parametrize("M,N,K,split", [(1280, 4000, 7168, 8), (2304, 3000, 12296, 2)])
def test_pair_kernel_split_tail(op, M, N, K, split):
    """More 256x256 tiles than clusters with a partly filled last round: with a scratch buffer the
    left-over tiles are cut along K (34 tiles in two parts, 6 tiles in eight parts, a ragged right
    edge and a ragged K) and finished by the tail reduce kernel; the contraction is long enough for
    the launcher to consider the split worth its reduce pass.  Same acceptance rule, identical bits on a rerun,
    ReLU / mask / overflow flag through the tail reduce, and the automatic choice takes the same path."""
    from paper_1710_03740_b200 import binding as b
    assert b.mpt_gemm_workspace_bytes(op, M, N, K) >= split * 256 * 256 * 4
    got, _, _, _ = _check_tc(op, M, N, K, workspace=True, kernel="pair")
    again, _, _, _ = _check_tc(op, M, N, K, workspace=True, kernel="pair")
    assert np.array_equal(got, again)
    auto, _, _, _ = _check_tc(op, M, N, K, workspace=True, kernel="auto")
    assert np.array_equal(got, auto)
    nows, _, _, _ = _check_tc(op, M, N, K, workspace=False, kernel="pair")       # half-width units instead
    assert (got != nows).mean() < 0.2                                            # same values up to summation order
    if split == 8:
        _check_tc(op, M, N, K, flags=b.GEMM_RELU, workspace=True, kernel="pair")
        mask = np.random.default_rng(8).standard_normal((M, N)).astype(np.float16)
        _check_tc(op, M, N, K, mask=mask, workspace=True, kernel="pair")
        _, ref, flag, _ = _check_tc(op, M, N, K, scale=30.0, want_flag=True, workspace=True, kernel="pair")
        assert flag == int(((ref & 0x7FFF) >= 0x7C00).any()) == 1


@pytest.mark.parametrize("op", [0, 1, 2])
def test_random_ragged_shapes_all_kernels(op):
    """Seeded random shapes with ragged M, N, K (pitches are multiples of 8): every kernel choice the
    library can make (single CTA, pair, automatic with and without a split-K workspace)."""
    from paper_1710_03740_b200 import binding as b
    rng = np.random.default_rng(1000 + op)
    for trial in range(14):
        M = int(rng.integers(1, 90)) * 8
        N = int(rng.integers(1, 90)) * 8
        K = int(rng.choice([8, 24, 64, 72, 200, 520, 1032, 2056, 4104]))
        relu = bool(rng.integers(0, 2))
        for kernel, ws in (("tc", False), ("pair", False), ("pair512", False), ("tc", True), ("pair", True), ("auto", True)):
            if ws and b.mpt_gemm_workspace_bytes(op, M, N, K) == 0:
                continue
            _check_tc(op, M, N, K, flags=b.GEMM_RELU if relu else 0, seed=int(rng.integers(1 << 30)), kernel=kernel,
                      workspace=ws)


@pytest.mark.parametrize("kernel", ["tc", "pair"])
def test_tc_gemm_relu_mask_flag_subnormals(kernel):
    from paper_1710_03740_b200 import binding as b
    M, N, K = 256, 512, 320
    _check_tc(0, M, N, K, flags=b.GEMM_RELU, kernel=kernel)
    rng = np.random.default_rng(4)
    mask = rng.standard_normal((M, N)).astype(np.float16)
    mask[0, :4] = [0.0, -0.0, np.nan, np.inf]
    _check_tc(1, M, N, K, mask=mask, kernel=kernel)
    # subnormal operands and outputs (config 2: head weights scaled by 2^-16)
    got, ref, _, stats = _check_tc(0, M, N, K, scale=2.0 ** -9, kernel=kernel)
    sub = (ref & 0x7C00) == 0
    assert sub.mean() > 0.5 and (ref[sub] != 0).any()
    # overflow on the store raises the flag (section 3.2)
    got, ref, flag, _ = _check_tc(2, M, N, K, scale=60.0, want_flag=True, kernel=kernel)
    assert flag == 1 and ((ref & 0x7FFF) == 0x7C00).any()
    got, ref, flag, _ = _check_tc(2, M, N, K, want_flag=True, kernel=kernel)
    assert flag == 0


def test_tc_gemm_rejects_unaligned():
    from paper_1710_03740_b200 import binding as b
    A = torch.zeros((16, 10), dtype=torch.int16, device="cuda")
    Bm = torch.zeros((16, 10), dtype=torch.int16, device="cuda")
    Cm = torch.zeros((16, 16), dtype=torch.int16, device="cuda")
    with pytest.raises(b.MptError) as e:
        b.mpt_gemm_f16(0, 16, 16, 10, A, 10, Bm, 10, Cm, 16, b.GEMM_FORCE_TC)
    assert e.value.code == -2
    b.mpt_gemm_f16(0, 16, 16, 10, A, 10, Bm, 10, Cm, 16, 0)     # falls back to the CUDA-core kernel
    torch.cuda.synchronize()
    with pytest.raises(b.MptError):
        b.mpt_gemm_f16(7, 16, 16, 10, A, 10, Bm, 10, Cm, 16, 0)
    with pytest.raises(b.MptError):
        b.mpt_gemm_f16(0, 16, 16, 10, A, 8, Bm, 10, Cm, 16, 0)  # pitch shorter than the row
