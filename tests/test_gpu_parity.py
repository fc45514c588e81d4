"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2608_10803_b200 import binding as ab
from paper_2608_10803_b200 import synth

from gpu_util import TOL, check_case, compare_with_oracle, init, run_library, sample_rows

pytestmark = pytest.mark.gpu

ROW, COL = ab.ROW_MAJOR, ab.COL_MAJOR


def draw(case):
    return synth.draw_case(case, device="cuda")


def every_variant(M, N, K, dtype, lA=ROW, lB=ROW, families=None, limit_per_family=40):
    """(plan, info) of every legal configuration, optionally restricted to some families."""
    out = []
    count = {}
    for c in ab.adapt_plan_candidates(M, N, K, dtype, lA, lB):
        if families is not None and c.family not in families:
            continue
        count[c.family] = count.get(c.family, 0) + 1
        if count[c.family] > limit_per_family:
            continue
        out.append((ab.adapt_matmul_plan_forced(M, N, K, dtype, lA, lB, c.tiling_key), c))
    return out


# ---- config 1: the 256^3 smoke case, full oracle, every variant ------------------------------------

def test_config1_square_256_all_variants():
    case = synth.config_square()[0]
    A, B = draw(case)
    for plan, c in every_variant(case.M, case.N, case.K, case.dtype):
        check_case(case.M, case.N, case.K, case.dtype, A, B, plan=plan)
    check_case(case.M, case.N, case.K, case.dtype, A, B)


# ---- exact cases: small integers, position-coded, bit-identical to the oracle ---------------------

EXACT_SHAPES = [
    (256, 256, 256), (200, 264, 328), (131, 77, 259), (128, 128, 64), (129, 65, 65), (1, 8, 8), (5, 640, 1000),
    (520, 3, 300), (16, 1024, 512), (1024, 16, 515), (300, 520, 8), (77, 50, 1), (384, 512, 2048), (64, 64, 8192),
]


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
@pytest.mark.parametrize("shape", EXACT_SHAPES)
def test_position_coded_integers_bit_exact_all_variants(shape, dtype):
    M, N, K = shape
    A = synth.position_coded(M, K, dtype, modulus=7, device="cuda")
    B = synth.position_coded(K, N, dtype, modulus=5, device="cuda").contiguous()
    for plan, c in every_variant(M, N, K, dtype, limit_per_family=12):
        check_case(M, N, K, dtype, A, B, plan=plan, exact=True)
    check_case(M, N, K, dtype, A, B, exact=True)


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
def test_random_integers_bit_exact(dtype):
    M, N, K = 300, 200, 1500
    A = synth.draw_operand(M, K, ("integer", -8, 8), 5, dtype, "cuda")
    B = synth.draw_operand(K, N, ("integer", -8, 8), 6, dtype, "cuda")
    for plan, c in every_variant(M, N, K, dtype, limit_per_family=6):
        check_case(M, N, K, dtype, A, B, plan=plan, exact=True)


# ---- layouts ------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
@pytest.mark.parametrize("lA,lB", [(ROW, COL), (COL, ROW), (COL, COL)])
@pytest.mark.parametrize("shape", [(256, 384, 512), (150, 90, 333), (8, 512, 640), (640, 8, 520)])
def test_layouts_bit_exact(shape, lA, lB, dtype):
    M, N, K = shape
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda")
    A_st = A.t().contiguous() if lA == COL else A       # column-major storage of A is A^T row-major
    B_st = B.t().contiguous() if lB == COL else B
    for plan, c in every_variant(M, N, K, dtype, lA, lB, limit_per_family=4):
        check_case(M, N, K, dtype, A_st, B_st, lA, lB, plan=plan, exact=True)


# ---- narrow operands: fewer than 64 contiguous elements, read over a copy with 32-byte rows ----------------

@pytest.mark.parametrize("lA,lB", [(ROW, ROW), (ROW, COL), (COL, ROW), (COL, COL)])
@pytest.mark.parametrize("shape", [(700, 520, 1), (700, 521, 8), (300, 40, 900), (1100, 5, 1300), (24, 300, 40), (9, 2100, 56),
                                   (1200, 84, 700), (2100, 330, 24)])
def test_narrow_operands_bit_exact(shape, lA, lB):
    """A, B (and through class tiles C) with rows of 2 to 126 bytes: every tensor-core configuration, among them
    class tiles over the re-pitched A and a B whose last box is a few columns wide, gives the oracle's bits."""
    M, N, K = shape
    dtype = ab.F16 if (M + N) % 2 == 0 else ab.BF16
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda")
    A_st = A.t().contiguous() if lA == COL else A
    B_st = B.t().contiguous() if lB == COL else B
    for plan, c in every_variant(M, N, K, dtype, lA, lB, families=(ab.FAM_UMMA_1CTA, ab.FAM_UMMA_2CTA), limit_per_family=10):
        check_case(M, N, K, dtype, A_st, B_st, lA, lB, plan=plan, exact=True)
    check_case(M, N, K, dtype, A_st, B_st, lA, lB, exact=True)


def test_narrow_operands_random_values_next_to_poisoned_memory():
    """The pad columns of the re-pitched copies hold zeros whatever follows the operands in memory: A and B sit in
    buffers whose other bytes are NaN patterns, and the result still meets the bar (a pad column that took a
    neighbour's value would put NaN into every output)."""
    for (M, N, K, dtype) in [(900, 5, 1500, ab.F16), (1300, 1031, 3, ab.BF16), (520, 40, 72, ab.F16)]:
        td = synth.torch_dtype(dtype)
        bufA = torch.full((M * K + 64,), float("nan"), dtype=td, device="cuda")
        bufB = torch.full((K * N + 64,), float("nan"), dtype=td, device="cuda")
        A = bufA[8:8 + M * K].view(M, K)
        B = bufB[8:8 + K * N].view(K, N)
        A.copy_(synth.draw_operand(M, K, synth.U11, 21, dtype, "cuda"))
        B.copy_(synth.draw_operand(K, N, synth.U11, 22, dtype, "cuda"))
        for plan, c in every_variant(M, N, K, dtype, families=(ab.FAM_UMMA_1CTA, ab.FAM_UMMA_2CTA), limit_per_family=6):
            check_case(M, N, K, dtype, A, B, plan=plan)


# ---- edge tiles: one off the tile sizes, primes, ones --------------------------------------------------

@pytest.mark.parametrize("shape", [(127, 255, 63), (129, 257, 65), (1, 1, 1), (2, 3, 5), (255, 129, 191),
                                   (128, 256, 64), (17, 1031, 257), (1031, 17, 129), (97, 89, 83)])
def test_edge_shapes_random_values(shape):
    M, N, K = shape
    for dtype in (ab.F16, ab.BF16):
        A = synth.draw_operand(M, K, synth.U11, 101, dtype, "cuda")
        B = synth.draw_operand(K, N, synth.U11, 102, dtype, "cuda")
        for plan, c in every_variant(M, N, K, dtype, limit_per_family=6):
            check_case(M, N, K, dtype, A, B, plan=plan)


def test_degenerate_sizes():
    init()
    dtype = ab.F16
    A = torch.ones((4, 0), dtype=torch.float16, device="cuda")
    B = torch.ones((0, 6), dtype=torch.float16, device="cuda")
    C = run_library(A, B, 4, 6, 0, dtype)                     # K = 0 -> zeros
    torch.cuda.synchronize()
    assert torch.count_nonzero(C).item() == 0 and not torch.isnan(C).any()
    run_library(torch.empty((0, 8), dtype=torch.float16, device="cuda"),
                torch.ones((8, 6), dtype=torch.float16, device="cuda"), 0, 6, 8, dtype)      # M = 0 -> no-op
    run_library(torch.ones((4, 8), dtype=torch.float16, device="cuda"),
                torch.empty((8, 0), dtype=torch.float16, device="cuda"), 4, 0, 8, dtype)      # N = 0 -> no-op
    torch.cuda.synchronize()


def test_argument_errors():
    init()
    h = ab.adapt_matmul_plan(64, 64, 64, ab.F16)
    A = torch.ones((64, 64), dtype=torch.float16, device="cuda")
    C = torch.empty((64, 64), dtype=torch.float16, device="cuda")
    with pytest.raises(ab.AdaptError) as e:
        ab.adapt_matmul(h, A.data_ptr(), A.data_ptr(), A.data_ptr(), 0)       # C aliases A
    assert e.value.status == ab.ERR_INVALID_ARG
    with pytest.raises(ab.AdaptError) as e:
        ab.adapt_matmul(h, 0, A.data_ptr(), C.data_ptr(), 0)
    assert e.value.status == ab.ERR_INVALID_ARG
    with pytest.raises(ab.AdaptError) as e:
        ab.adapt_matmul(h, A.data_ptr() + 1, A.data_ptr(), C.data_ptr(), 0)   # odd address
    assert e.value.status == ab.ERR_INVALID_ARG


def test_misaligned_pointers_take_the_repitch_path():
    """Buffers that start 2 bytes off a 16-byte boundary still give the exact result."""
    M, N, K = 256, 256, 512
    dtype = ab.BF16
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda")
    bufA = torch.zeros(M * K + 8, dtype=torch.bfloat16, device="cuda")
    bufB = torch.zeros(K * N + 8, dtype=torch.bfloat16, device="cuda")
    bufC = torch.zeros(M * N + 8, dtype=torch.bfloat16, device="cuda")
    A1 = bufA[1:1 + M * K].view(M, K)
    B1 = bufB[3:3 + K * N].view(K, N)
    C1 = bufC[5:5 + M * N].view(M, N)
    A1.copy_(A)
    B1.copy_(B)
    for plan, c in every_variant(M, N, K, dtype, limit_per_family=3):
        C1.fill_(float("nan"))
        run_library(A1, B1, M, N, K, dtype, plan=plan, out=C1)
        torch.cuda.synchronize()
        err, mism, n = compare_with_oracle(A1, B1, C1, M, N, K, dtype)
        assert mism == 0, (ab.FAMILY_NAMES[c.family], c.BN, c.P_k, mism)
    assert bufC[:5].abs().sum().item() == 0 and bufC[5 + M * N:].abs().sum().item() == 0   # no stray writes


def test_run_twice_is_bit_identical():
    for (M, N, K, dtype) in [(256, 256, 262144 // 8, ab.BF16), (7, 1024, 1024, ab.F16), (1000, 1024, 1024, ab.F16)]:
        A = synth.draw_operand(M, K, synth.U11, 1, dtype, "cuda")
        B = synth.draw_operand(K, N, synth.U11, 2, dtype, "cuda")
        for plan, c in every_variant(M, N, K, dtype, limit_per_family=3):
            C1 = run_library(A, B, M, N, K, dtype, plan=plan).clone()
            C2 = run_library(A, B, M, N, K, dtype, plan=plan)
            torch.cuda.synchronize()
            assert torch.equal(C1.view(torch.int16), C2.view(torch.int16))


# ---- the named workloads at full size, in the configuration bench.py times (model-selected plan) ----

@pytest.mark.parametrize("case", synth.config_reco(), ids=lambda c: c.name)
def test_config2_recommendation_shapes(case):
    A, B = draw(case)
    check_case(case.M, case.N, case.K, case.dtype, A, B, mac_budget=3e9)


@pytest.mark.parametrize("case", synth.config_llm(), ids=lambda c: c.name)
def test_config3_llm_layer_shapes(case):
    A, B = draw(case)
    check_case(case.M, case.N, case.K, case.dtype, A, B, mac_budget=1.5e10)


@pytest.mark.parametrize("case", synth.config_large(), ids=lambda c: c.name)
def test_config4_large_and_tall_k(case):
    A, B = draw(case)
    check_case(case.M, case.N, case.K, case.dtype, A, B, mac_budget=1.8e10)


@pytest.mark.parametrize("case", synth.config_context(), ids=lambda c: c.name)
def test_paper_named_shapes(case):
    A, B = draw(case)
    check_case(case.M, case.N, case.K, case.dtype, A, B, mac_budget=6e9)


def test_sweep_oracle_subset():
    """The seeded 200-shape subset of the 2,000-shape dynamic sweep; complete sampled rows on the
    larger shapes so the CPU side stays within a minute or two."""
    cases = synth.config_sweep()
    worst = {ab.F16: 0.0, ab.BF16: 0.0}
    for idx in synth.sweep_oracle_subset():
        case = cases[idx]
        A, B = draw(case)
        err, _, _, _ = check_case(case.M, case.N, case.K, case.dtype, A, B, mac_budget=4e8, seed=idx)
        worst[case.dtype] = max(worst[case.dtype], err)
        del A, B
    assert worst[ab.F16] <= TOL[ab.F16] and worst[ab.BF16] <= TOL[ab.BF16]


def test_long_k_accumulation_error_stays_small():
    """fp32 accumulation over a very long chain (no split): error must stay far below tolerance."""
    M, N, K = 128, 128, 131072
    dtype = ab.BF16
    A = synth.draw_operand(M, K, synth.U11, 7, dtype, "cuda")
    B = synth.draw_operand(K, N, synth.U11, 8, dtype, "cuda")
    for plan, c in every_variant(M, N, K, dtype, families=[ab.FAM_UMMA_1CTA]):
        if c.P_k != 1 or c.BN != 128:
            continue
        err, _, _, _ = check_case(M, N, K, dtype, A, B, plan=plan)
        assert err < 4e-3


# ---- row-major A with K % 8 != 0 read in place through per-row-class TMA views --------------------

def class_mode_variants(M, N, K, dtype, limit=6):
    out = []
    for c in ab.adapt_plan_candidates(M, N, K, dtype):
        if c.srcA == 3 and len(out) < limit:
            out.append((ab.adapt_matmul_plan_forced(M, N, K, dtype, ROW, ROW, c.tiling_key), c))
    return out


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
@pytest.mark.parametrize("shape", [(131, 77, 259), (1030, 264, 331), (2500, 64, 1001), (8, 8, 9), (300, 520, 12),
                                   (1024, 128, 4099), (77, 1000, 70), (4100, 16, 2047)])
def test_row_class_views_bit_exact(shape, dtype):
    M, N, K = shape
    A = synth.position_coded(M, K, dtype, modulus=7, device="cuda")
    B = synth.position_coded(K, N, dtype, modulus=5, device="cuda")
    variants = class_mode_variants(M, N, K, dtype)
    assert variants, "shape must offer the class-mode source for A"
    for plan, c in variants:
        check_case(M, N, K, dtype, A, B, plan=plan, exact=True)


def test_row_class_views_do_not_leak_a_neighbouring_row():
    """The elements in front of a class row's first element belong to the previous row of A; a
    non-finite value there must not reach this row's result."""
    M, N, K = 600, 136, 203
    dtype = ab.F16
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda")
    bad_rows = [4, 17, 300]
    for r in bad_rows:
        A[r, K - 1] = float("inf")            # the tail of row r precedes the head of row r + 1 in memory
        A[r, K - 2] = float("nan")
    keep = torch.tensor([i for i in range(M) if i not in bad_rows], device="cuda")
    for plan, c in class_mode_variants(M, N, K, dtype):
        C = run_library(A, B, M, N, K, dtype, plan=plan)
        torch.cuda.synchronize()
        assert torch.isfinite(C.index_select(0, keep)).all()
        err, mism, n = compare_with_oracle(A, B, C, M, N, K, dtype, rows=keep.cpu().numpy())
        assert mism == 0


# ---- row-major B with N % 8 != 0 read in place through per-k-class TMA views ----------------------

def kclass_mode_variants(M, N, K, dtype, layoutA=ROW, limit=4):
    """Up to `limit` variants each of the two forms: eight class accumulators per tile (BN = 64) and
    classes as k splits (BN = 128, 256)."""
    cands = [c for c in ab.adapt_plan_candidates(M, N, K, dtype, layoutA, ROW) if c.srcB == 3]
    picked = [c for c in cands if c.BN == 64][:limit]
    split = [c for c in cands if c.BN != 64]
    one = [c for c in split if c.family == ab.FAM_UMMA_1CTA]
    pair = [c for c in split if c.family == ab.FAM_UMMA_2CTA]
    for group in (one, pair):
        picked += [c for c in group if c.P_k == 8][: limit // 2] + [c for c in group if c.P_k > 8][: limit // 2]
    return [(ab.adapt_matmul_plan_forced(M, N, K, dtype, layoutA, ROW, c.tiling_key), c) for c in picked]


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
@pytest.mark.parametrize("shape", [(8, 3001, 4000), (100, 777, 1000), (131, 57, 64), (17, 55, 1031), (300, 9, 70),
                                   (129, 1234, 513), (5, 113, 5003), (64, 20002, 300)])
def test_k_class_views_bit_exact(shape, dtype):
    M, N, K = shape
    A = synth.position_coded(M, K, dtype, modulus=7, device="cuda")
    B = synth.position_coded(K, N, dtype, modulus=5, device="cuda")
    variants = kclass_mode_variants(M, N, K, dtype)
    assert variants, "shape must offer the k-class source for B"
    assert any(c.P_k > 1 for _, c in variants) or K < 1024
    assert any(c.BN != 64 and c.family == ab.FAM_UMMA_1CTA for _, c in variants), "classes as k splits must be on offer"
    assert any(c.family == ab.FAM_UMMA_2CTA for _, c in variants), "... and on pair tiles"
    for plan, c in variants:
        check_case(M, N, K, dtype, A, B, plan=plan, exact=True)


def test_k_class_views_with_column_major_a_and_random_values():
    M, N, K = 77, 1001, 2049
    for dtype in (ab.F16, ab.BF16):
        A = synth.draw_operand(K, M, synth.U11, 21, dtype, "cuda")      # storage of a column-major A
        B = synth.draw_operand(K, N, synth.U11, 22, dtype, "cuda")
        variants = kclass_mode_variants(M, N, K, dtype, layoutA=COL)
        assert variants
        for plan, c in variants:
            err, _, _, _ = check_case(M, N, K, dtype, A, B, COL, ROW, plan=plan)
            assert err <= TOL[dtype]


def test_k_class_views_do_not_leak_a_neighbouring_row():
    """The elements in front of a class row's first element belong to the previous row of B; they land
    in accumulator columns that are never read, so a non-finite value in column N - 1 of a row of B may
    only reach column N - 1 of the result."""
    M, N, K = 40, 203, 600
    dtype = ab.F16
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda")
    ref = run_library(A, B, M, N, K, dtype).clone()                 # checked against the oracle below
    err, mism, _ = compare_with_oracle(A, B, ref, M, N, K, dtype)
    assert mism == 0
    for r in (4, 17, 300):
        B[r, N - 1] = float("inf")
    variants = kclass_mode_variants(M, N, K, dtype)
    assert variants
    for plan, c in variants:
        C = run_library(A, B, M, N, K, dtype, plan=plan)
        torch.cuda.synchronize()
        assert torch.isfinite(C[:, : N - 1]).all()
        assert torch.equal(synth_bits(C[:, : N - 1]), synth_bits(ref[:, : N - 1]))


def synth_bits(t):
    return t.contiguous().view(torch.int16)


# ---- class tiles with halo columns: C with N % 8 != 0 written through per-row-class TMA stores ------

def halo_variants(M, N, K, dtype, limit=12, family=None):
    """Class tiles with halo columns: for every kernel family and tile width on offer, the best variant that stores
    C itself (P_k = 1, the TMA-store epilogue) and the best one that writes fp32 partials."""
    cands = [c for c in ab.adapt_plan_candidates(M, N, K, dtype) if c.srcA == 3 and c.BN % 64 != 0
             and (family is None or c.family == family)]
    picked = []
    for fam, bn in sorted({(c.family, c.BN) for c in cands}):
        mine = [c for c in cands if c.BN == bn and c.family == fam]
        picked += [c for c in mine if c.P_k == 1][:1] + [c for c in mine if c.P_k > 1][:1]
    return [(ab.adapt_matmul_plan_forced(M, N, K, dtype, ROW, ROW, c.tiling_key), c) for c in picked[:limit]]


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
@pytest.mark.parametrize("shape", [(1030, 265, 328), (1030, 265, 331), (2500, 77, 1000), (4100, 1001, 64), (300, 521, 16),
                                   (16, 9, 8), (129, 3, 40), (1024, 201, 4099), (3000, 40, 24), (2100, 8, 16), (77, 1537, 70), (2049, 193, 5),
                                   # even N: 8, 4 or 2 row classes instead of 16 (and what an A read in place adds to that)
                                   (1030, 266, 331), (1030, 268, 328), (4100, 1000, 64), (2049, 200, 5), (300, 518, 20), (2100, 12, 16),
                                   (999, 36, 100), (1500, 104, 70), (5000, 1032, 257)])
def test_halo_class_tiles_bit_exact(shape, dtype):
    M, N, K = shape
    A = synth.position_coded(M, K, dtype, modulus=7, device="cuda")
    B = synth.position_coded(K, N, dtype, modulus=5, device="cuda")
    variants = halo_variants(M, N, K, dtype)
    assert variants, "shape must offer class tiles with halo columns"
    assert {c.BN for _, c in variants} == {80, 144, 208}
    for plan, c in variants:
        check_case(M, N, K, dtype, A, B, plan=plan, exact=True)


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
@pytest.mark.parametrize("shape", [(1030, 265, 328), (1030, 265, 331), (4100, 1001, 64), (300, 521, 16), (40, 777, 200),
                                   (4097, 201, 1003), (9000, 393, 24), (2100, 209, 700), (8200, 1537, 70), (5000, 193, 5),
                                   (4097, 204, 1003), (9000, 392, 24), (2100, 210, 700), (1100, 1000, 72)])
def test_pair_halo_class_tiles_bit_exact(shape, dtype):
    """Halo class tiles on SM pairs (256 rows of one of 16 row classes, 128 or 192 owned columns + 16 halo columns):
    aligned and unaligned A, K shorter and longer than a k-block, M below and above one group of 4096 rows,
    with the TMA-store epilogue and with fp32 partials, against the oracle on position-coded integers."""
    M, N, K = shape
    A = synth.position_coded(M, K, dtype, modulus=7, device="cuda")
    B = synth.position_coded(K, N, dtype, modulus=5, device="cuda")
    variants = halo_variants(M, N, K, dtype, family=ab.FAM_UMMA_2CTA)
    assert variants and {c.BN for _, c in variants} == {144, 208}
    for plan, c in variants:
        check_case(M, N, K, dtype, A, B, plan=plan, exact=True)


def test_pair_halo_class_tiles_random_values_and_guard_bands():
    """Random values, C inside a buffer whose other bytes must stay as they were (the per-class TMA stores and the
    narrow stores at the row ends write nothing beyond row M - 1 or column N - 1)."""
    for (M, N, K, dtype) in [(2300, 1001, 520, ab.F16), (4200, 265, 40, ab.BF16)]:
        A = synth.draw_operand(M, K, synth.U11, 31, dtype, "cuda")
        B = synth.draw_operand(K, N, synth.U11, 32, dtype, "cuda")
        guard = 4096
        buf = torch.full((M * N + 2 * guard,), 77.0, dtype=A.dtype, device="cuda")
        C = buf[guard:guard + M * N].view(M, N)
        for plan, c in halo_variants(M, N, K, dtype, family=ab.FAM_UMMA_2CTA):
            buf.fill_(77.0)
            run_library(A, B, M, N, K, dtype, plan=plan, out=C)
            torch.cuda.synchronize()
            ab.adapt_poll_device_status(torch.cuda.current_stream().cuda_stream)
            assert bool((buf[:guard] == 77.0).all()) and bool((buf[guard + M * N:] == 77.0).all())
            err, mism, n = compare_with_oracle(A, B, C, M, N, K, dtype)
            assert err <= TOL[dtype], (M, N, K, c.BN, c.P_k, err)


def test_halo_class_tiles_with_unaligned_pointers():
    """A or C two bytes off a 16-byte boundary: A is then read through a re-pitched copy, C is stored by
    the epilogue threads; the tiling stays the plan's."""
    M, N, K = 1100, 333, 203
    dtype = ab.F16
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda")
    tdt = synth.torch_dtype(dtype)
    a_buf = torch.zeros(M * K + 16, dtype=tdt, device="cuda")
    A_off = a_buf[1:1 + M * K].view(M, K)
    A_off.copy_(A)
    assert A_off.data_ptr() % 16 == 2
    variants = halo_variants(M, N, K, dtype, limit=4)
    assert variants
    for plan, c in variants:
        for a_t, c_off in ((A_off, 0), (A, 1), (A_off, 1)):
            c_buf = torch.full((M * N + 16,), float("nan"), dtype=tdt, device="cuda")
            out = c_buf[c_off:c_off + M * N].view(M, N)
            run_library(a_t, B, M, N, K, dtype, plan=plan, out=out)
            torch.cuda.synchronize()
            err, mism, _ = compare_with_oracle(A, B, out.contiguous(), M, N, K, dtype)
            assert mism == 0
            # nothing outside C was touched
            assert torch.isnan(c_buf[:c_off]).all() and torch.isnan(c_buf[c_off + M * N:]).all()


def test_tma_store_epilogue_leaves_neighbouring_memory_alone():
    """Aligned and halo TMA stores clip at M and at the end of each row: guard elements around C stay."""
    dtype = ab.BF16
    tdt = synth.torch_dtype(dtype)
    for (M, N, K) in [(200, 264, 64), (1031, 203, 72), (130, 72, 40)]:
        A = synth.position_coded(M, K, dtype, 7, "cuda")
        B = synth.position_coded(K, N, dtype, 5, "cuda")
        c_buf = torch.full((M * N + 4096,), float("nan"), dtype=tdt, device="cuda")
        out = c_buf[2048:2048 + M * N].view(M, N)
        assert out.data_ptr() % 16 == 0
        run_library(A, B, M, N, K, dtype, out=out)
        torch.cuda.synchronize()
        err, mism, _ = compare_with_oracle(A, B, out.contiguous(), M, N, K, dtype)
        assert mism == 0
        assert torch.isnan(c_buf[:2048]).all() and torch.isnan(c_buf[2048 + M * N:]).all()


# ---- the one-launch cluster kernel: every cluster size, layout and alignment ---------------------------------

def cluster_variants(M, N, K, dtype, lA=ROW, lB=ROW):
    cands = [c for c in ab.adapt_plan_candidates(M, N, K, dtype, lA, lB) if c.family == ab.FAM_CLUSTER]
    return [(ab.adapt_matmul_plan_forced(M, N, K, dtype, lA, lB, c.tiling_key), c) for c in cands]


@pytest.mark.parametrize("lA,lB", [(ROW, ROW), (ROW, COL), (COL, ROW), (COL, COL)])
@pytest.mark.parametrize("shape", [(64, 64, 64), (70, 130, 100), (200, 333, 1482), (129, 65, 17), (33, 7, 4099),
                                   (1, 1, 1), (300, 264, 520), (3, 200, 129), (65, 63, 8)])
def test_cluster_family_bit_exact(shape, lA, lB):
    M, N, K = shape
    for dtype in (ab.F16, ab.BF16):
        A = synth.position_coded(M, K, dtype, 7, "cuda")
        B = synth.position_coded(K, N, dtype, 5, "cuda")
        A_st = A.t().contiguous() if lA == COL else A
        B_st = B.t().contiguous() if lB == COL else B
        variants = cluster_variants(M, N, K, dtype, lA, lB)
        assert any(c.cluster == 1 and c.P_k == 1 for _, c in variants)
        # every cluster size that leaves no CTA without k values (pieces are multiples of 16)
        want = {cs for cs in (1, 2, 4, 8, 16) if (cs - 1) * (-(-(-(-K // cs)) // 16) * 16) < K
                and cs * (-(-M // 64)) * (-(-N // 64)) <= 2 * 148}
        assert {c.cluster for _, c in variants} == want
        for plan, c in variants:
            assert c.P_k == c.cluster and c.workspace_bytes == 0
            check_case(M, N, K, dtype, A_st, B_st, lA, lB, plan=plan, exact=True)


def test_cluster_family_random_values_and_unaligned_pointers():
    """Operands and C two bytes off a 16-byte boundary (rows of aligned pitch, misaligned base): the groups
    are then assembled from two chunks; nothing outside C is written."""
    M, N, K = 150, 200, 328
    dtype = ab.BF16
    tdt = synth.torch_dtype(dtype)
    A = synth.draw_operand(M, K, synth.U11, 31, dtype, "cuda")
    B = synth.draw_operand(K, N, synth.U11, 32, dtype, "cuda")
    a_buf = torch.zeros(M * K + 16, dtype=tdt, device="cuda")
    b_buf = torch.zeros(K * N + 16, dtype=tdt, device="cuda")
    A_off = a_buf[1:1 + M * K].view(M, K)
    B_off = b_buf[3:3 + K * N].view(K, N)
    A_off.copy_(A)
    B_off.copy_(B)
    assert A_off.data_ptr() % 16 == 2 and B_off.data_ptr() % 16 == 6
    for plan, c in cluster_variants(M, N, K, dtype):
        for a_t, b_t, c_off in ((A, B, 0), (A_off, B, 1), (A, B_off, 0), (A_off, B_off, 3)):
            c_buf = torch.full((M * N + 16,), float("nan"), dtype=tdt, device="cuda")
            out = c_buf[c_off:c_off + M * N].view(M, N)
            run_library(a_t, b_t, M, N, K, dtype, plan=plan, out=out)
            torch.cuda.synchronize()
            err, mism, _ = compare_with_oracle(A, B, out.contiguous(), M, N, K, dtype)
            assert err <= 8e-3
            assert torch.isnan(c_buf[:c_off]).all() and torch.isnan(c_buf[c_off + M * N:]).all()


# ---- host operands: the pipelined copy-in | kernels | copy-out entry point ------------------------------

def test_host_entry_point_matches_the_oracle_over_a_run_of_calls():
    """Seven calls back to back on one stream (both staging slots reused several times, growing and
    shrinking shapes, both dtypes), results read only after one synchronisation at the end."""
    shapes = [(131, 77, 259, ab.F16), (1030, 265, 331, ab.BF16), (8, 3001, 400, ab.F16), (256, 256, 256, ab.BF16),
              (5, 640, 1000, ab.F16), (2049, 193, 5, ab.BF16), (300, 520, 12, ab.F16)]
    st = torch.cuda.current_stream().cuda_stream
    jobs = []
    for (M, N, K, dtype) in shapes:
        A = synth.position_coded(M, K, dtype, 7, "cpu").pin_memory()
        B = synth.position_coded(K, N, dtype, 5, "cpu").pin_memory()
        C = torch.full((M, N), float("nan"), dtype=synth.torch_dtype(dtype)).pin_memory()
        plan = ab.adapt_matmul_plan(M, N, K, dtype)
        ab.adapt_matmul_host(plan, A.data_ptr(), B.data_ptr(), C.data_ptr(), st)
        jobs.append((M, N, K, dtype, A, B, C))
    torch.cuda.synchronize()
    ab.adapt_poll_device_status(st)
    for (M, N, K, dtype, A, B, C) in jobs:
        err, mism, _ = compare_with_oracle(A, B, C, M, N, K, dtype)
        assert mism == 0, (M, N, K)


def test_host_entry_point_twice_is_bit_identical_and_orders_the_callers_stream():
    M, N, K, dtype = 777, 1001, 513, ab.BF16
    A = synth.draw_operand(M, K, synth.U11, 5, dtype, "cpu").pin_memory()
    B = synth.draw_operand(K, N, synth.U11, 6, dtype, "cpu").pin_memory()
    C1 = torch.zeros((M, N), dtype=synth.torch_dtype(dtype)).pin_memory()
    C2 = torch.zeros((M, N), dtype=synth.torch_dtype(dtype)).pin_memory()
    plan = ab.adapt_matmul_plan(M, N, K, dtype)
    s = torch.cuda.Stream()
    ab.adapt_matmul_host(plan, A.data_ptr(), B.data_ptr(), C1.data_ptr(), s.cuda_stream)
    ab.adapt_matmul_host(plan, A.data_ptr(), B.data_ptr(), C2.data_ptr(), s.cuda_stream)
    s.synchronize()                       # the caller's stream alone: it waits for both copies of C
    assert torch.equal(C1.view(torch.int16), C2.view(torch.int16))
    err, _, _ = compare_with_oracle(A, B, C1, M, N, K, dtype)
    assert err <= TOL[dtype]


# ---- plan-cache key beyond the packed range; tensor-map cache; the bounded-wait path ----------------------

@pytest.mark.parametrize("shape", [((1 << 20) + 3, 8, 24), (16, (1 << 20) + 8, 40), (9, 24, (1 << 20) + 5)])
def test_dimension_beyond_the_packed_shape_key(shape):
    """A dimension of 2^20 or more does not fit the packed 64-bit shape word: the plan comes from the slow-path
    table, is still cached (same handle) and runs like any other."""
    M, N, K = shape
    dtype = ab.BF16
    init()
    h1 = ab.adapt_matmul_plan(M, N, K, dtype)
    h2 = ab.adapt_matmul_plan(M, N, K, dtype)
    assert h1 == h2
    A = synth.draw_operand(M, K, ("integer", -3, 3), 31, dtype, "cuda")
    B = synth.draw_operand(K, N, ("integer", -3, 3), 32, dtype, "cuda")
    check_case(M, N, K, dtype, A, B, plan=h1, exact=True, mac_budget=2e9)


def test_tensor_map_cache_keeps_geometries_apart():
    """One plan can reach the same workspace address with two tile geometries: a k-class plan (B read in place
    through per-class views, A regrouped into the workspace) falls back to re-pitched copies when B's pointer
    is not 16-byte aligned, and with a column-major A the two layouts of the workspace copy of A can share
    base pointer and pitch.  The cache must not hand the map of one to the other, in either order."""
    M, K, N = 510, 260, 1003                 # padded_pitch(M) = 512 = 8 * Kc with Kc = 64 ... checked below
    dtype = ab.F16
    init()
    cands = [c for c in ab.adapt_plan_candidates(M, N, K, dtype, COL, ROW) if c.srcB == 3]
    assert cands, "expected a k-class configuration for this shape"
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda")
    A_st = A.t().contiguous()
    bufB = torch.zeros(K * N + 8, dtype=torch.float16, device="cuda")
    B_off = bufB[1:1 + K * N].view(K, N)
    B_off.copy_(B)
    for c in cands[:3]:
        plan = ab.adapt_matmul_plan_forced(M, N, K, dtype, COL, ROW, c.tiling_key)
        for order in ((B, B_off, B), (B_off, B, B_off)):
            for Bx in order:
                C = run_library(A_st, Bx, M, N, K, dtype, COL, ROW, plan=plan)
                torch.cuda.synchronize()
                ab.adapt_poll_device_status(torch.cuda.current_stream().cuda_stream)
                err, mism, n = compare_with_oracle(A_st, Bx, C, M, N, K, dtype, COL, ROW)
                assert mism == 0, (c.BN, c.P_k, mism)


def test_tensor_map_cache_hits_after_the_first_call_and_holds_eight_pointer_sets():
    init()
    M, N, K, dtype = 512, 512, 512, ab.BF16
    plan = ab.adapt_matmul_plan(M, N, K, dtype)
    st = torch.cuda.current_stream().cuda_stream
    sets = [(synth.draw_operand(M, K, synth.U11, 40 + i, dtype, "cuda"), synth.draw_operand(K, N, synth.U11, 60 + i, dtype, "cuda"),
             torch.empty((M, N), dtype=torch.bfloat16, device="cuda")) for i in range(8)]
    for a, b, c in sets:
        ab.adapt_matmul(plan, a.data_ptr(), b.data_ptr(), c.data_ptr(), st)
    before = ab.adapt_map_encode_count()
    for _ in range(3):
        for a, b, c in sets:
            ab.adapt_matmul(plan, a.data_ptr(), b.data_ptr(), c.data_ptr(), st)
    torch.cuda.synchronize()
    assert ab.adapt_map_encode_count() == before, "a rotation over eight pointer sets must not encode a tensor map"
    ref = sets[0][2].clone()
    ab.adapt_set_map_cache(False)
    try:
        ab.adapt_matmul(plan, sets[0][0].data_ptr(), sets[0][1].data_ptr(), sets[0][2].data_ptr(), st)
        torch.cuda.synchronize()
        assert ab.adapt_map_encode_count() > before
    finally:
        ab.adapt_set_map_cache(True)
    assert torch.equal(ref.view(torch.int16), sets[0][2].view(torch.int16))


def test_bounded_wait_expires_and_reports_a_timeout():
    """A wait on a barrier nobody arrives on gives up after its limit: the kernel ends normally, the status word
    is set, the poll reports ADAPT_ERR_TIMEOUT once, and the library keeps working afterwards."""
    init()
    st = torch.cuda.current_stream().cuda_stream
    ab.adapt_poll_device_status(st)                       # clean to begin with
    ab.adapt_selftest_wait_expiry(1_000_000, st)          # 1 ms
    with pytest.raises(ab.AdaptError) as e:
        ab.adapt_poll_device_status(st)
    assert e.value.status == ab.ERR_TIMEOUT
    ab.adapt_poll_device_status(st)                       # the word was cleared by the failing poll
    M, N, K, dtype = 256, 256, 256, ab.F16
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda")
    check_case(M, N, K, dtype, A, B, exact=True)


def test_batch_of_many_calls_on_internal_streams_matches_single_calls_and_keeps_dependences():
    """A batch long enough for the internal streams of the batch entry: 40 independent calls of mixed shapes (stream-K, fused and
    class-tile plans among them) give the bits of the same calls made one by one; then a chain inside one batch, every
    call reading the output of the one before and the last overwriting the first one's output, gives what the chain gives
    call by call (the batch entry orders calls whose buffers overlap)."""
    init()
    st = torch.cuda.current_stream().cuda_stream
    base = [(131, 77, 259, ab.BF16), (512, 512, 2048, ab.BF16), (8, 3001, 400, ab.F16), (300, 520, 12, ab.F16), (2560, 2048, 2048, ab.F16),
            (1, 4096, 4096, ab.BF16), (1030, 265, 331, ab.F16), (64, 64, 8192, ab.F16), (5, 640, 1000, ab.BF16), (2049, 128, 4099, ab.F16)]
    shapes = [base[i % len(base)] for i in range(40)]
    plans, As, Bs, C1, C2 = [], [], [], [], []
    for i, (M, N, K, dt) in enumerate(shapes):
        plans.append(ab.adapt_matmul_plan(M, N, K, dt))
        As.append(synth.draw_operand(M, K, synth.U11, 170 + i, dt, "cuda"))
        Bs.append(synth.draw_operand(K, N, synth.U11, 290 + i, dt, "cuda"))
        C1.append(torch.full((M, N), float("nan"), dtype=As[-1].dtype, device="cuda"))
        C2.append(torch.full((M, N), float("nan"), dtype=As[-1].dtype, device="cuda"))
    for p, a, b, c in zip(plans, As, Bs, C1):
        ab.adapt_matmul(p, a.data_ptr(), b.data_ptr(), c.data_ptr(), st)
    for _ in range(2):
        ab.adapt_matmul_batch(plans, [a.data_ptr() for a in As], [b.data_ptr() for b in Bs], [c.data_ptr() for c in C2], st)
    torch.cuda.synchronize()
    ab.adapt_poll_device_status(st)
    for c1, c2 in zip(C1, C2):
        assert torch.equal(c1.view(torch.int16), c2.view(torch.int16))
    # a chain: X_{i+1} = X_i * W_i (square, small integers keep the values exact in fp16 for a while), in one batch
    n, links = 256, 12
    plan = ab.adapt_matmul_plan(n, n, n, ab.F16)
    X0 = synth.position_coded(n, n, ab.F16, 3, "cuda")
    eye = torch.eye(n, dtype=torch.float16, device="cuda")
    Ws = [(eye + (torch.roll(eye, i + 1, 1) if i % 2 else 0)).contiguous() for i in range(links)]     # permutation-like, entries 0/1
    def run(batch):
        X = [X0.clone()] + [torch.full((n, n), float("nan"), dtype=torch.float16, device="cuda") for _ in range(links - 1)]
        outs = X[1:] + [X[0]]                      # the last link writes over the first buffer
        ins = [X[0]] + X[1:]
        # link 0 reads X[0]; the last link writes X[0]: it must wait for link 0 as well as for its own input
        ins = [X[i] for i in range(links)]
        if batch:
            ab.adapt_matmul_batch([plan] * links, [t.data_ptr() for t in ins], [w.data_ptr() for w in Ws], [t.data_ptr() for t in outs], st)
        else:
            for a, w, c in zip(ins, Ws, outs):
                ab.adapt_matmul(plan, a.data_ptr(), w.data_ptr(), c.data_ptr(), st)
        torch.cuda.synchronize()
        return [t.clone() for t in X]
    ref, got = run(False), run(True)
    for r, g in zip(ref, got):
        assert not torch.isnan(g).any() and torch.equal(r.view(torch.int16), g.view(torch.int16))


def test_batch_entry_can_be_captured_into_a_cuda_graph_and_replayed():
    """After a warm-up call (workspaces grown, tensor maps cached) the batch entry only launches kernels and records
    and waits for events, so a stream capture takes it, internal streams included; replays give the bits of the direct
    calls, also after the inputs change in place."""
    init()
    shapes = [(131, 77, 259, ab.BF16), (512, 512, 2048, ab.BF16), (8, 3001, 400, ab.F16), (300, 520, 12, ab.F16), (1030, 265, 331, ab.F16),
              (64, 64, 8192, ab.F16), (5, 640, 1000, ab.BF16), (1, 4096, 4096, ab.BF16), (200, 264, 328, ab.F16), (77, 50, 1, ab.F16)]
    plans, As, Bs, Cd, Cg = [], [], [], [], []
    for i, (M, N, K, dt) in enumerate(shapes):
        plans.append(ab.adapt_matmul_plan(M, N, K, dt))
        As.append(synth.draw_operand(M, K, synth.U11, 400 + i, dt, "cuda"))
        Bs.append(synth.draw_operand(K, N, synth.U11, 500 + i, dt, "cuda"))
        Cd.append(torch.full((M, N), float("nan"), dtype=As[-1].dtype, device="cuda"))
        Cg.append(torch.full((M, N), float("nan"), dtype=As[-1].dtype, device="cuda"))
    pa, pb = ab.pointer_array([t.data_ptr() for t in As]), ab.pointer_array([t.data_ptr() for t in Bs])
    pd, pg, pp = ab.pointer_array([t.data_ptr() for t in Cd]), ab.pointer_array([t.data_ptr() for t in Cg]), ab.pointer_array(plans)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(2):
            ab.adapt_matmul_batch(pp, pa, pb, pg, side.cuda_stream)          # warm-up on the capturing stream
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            ab.adapt_matmul_batch(pp, pa, pb, pg, side.cuda_stream)
    torch.cuda.synchronize()
    st = torch.cuda.current_stream().cuda_stream
    for round_ in range(2):
        for c in Cg:
            c.fill_(float("nan"))
        torch.cuda.synchronize()
        graph.replay()
        ab.adapt_matmul_batch(pp, pa, pb, pd, st)
        torch.cuda.synchronize()
        ab.adapt_poll_device_status(st)
        for cd, cg in zip(Cd, Cg):
            assert not torch.isnan(cg).any() and torch.equal(cd.view(torch.int16), cg.view(torch.int16))
        for a in As:                                  # new contents, same buffers: the replay must follow
            a.mul_(-0.5)


def test_batched_entry_point_matches_single_calls():
    init()
    st = torch.cuda.current_stream().cuda_stream
    shapes = [(131, 77, 259, ab.BF16), (512, 512, 2048, ab.BF16), (8, 3001, 400, ab.F16), (1, 1, 1, ab.F16), (300, 520, 12, ab.F16)]
    plans, As, Bs, C1, C2 = [], [], [], [], []
    for i, (M, N, K, dt) in enumerate(shapes):
        plans.append(ab.adapt_matmul_plan(M, N, K, dt))
        As.append(synth.draw_operand(M, K, synth.U11, 70 + i, dt, "cuda"))
        Bs.append(synth.draw_operand(K, N, synth.U11, 90 + i, dt, "cuda"))
        C1.append(torch.full((M, N), float("nan"), dtype=As[-1].dtype, device="cuda"))
        C2.append(torch.full((M, N), float("nan"), dtype=As[-1].dtype, device="cuda"))
        ab.adapt_matmul(plans[-1], As[-1].data_ptr(), Bs[-1].data_ptr(), C1[-1].data_ptr(), st)
    ab.adapt_matmul_batch(plans, [a.data_ptr() for a in As], [b.data_ptr() for b in Bs], [c.data_ptr() for c in C2], st)
    ab.adapt_matmul_repeat(plans[0], [As[0].data_ptr()] * 2, [Bs[0].data_ptr()] * 2, [C2[0].data_ptr()] * 2, 3, st)
    torch.cuda.synchronize()
    ab.adapt_poll_device_status(st)
    for a, b in zip(C1, C2):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    (M, N, K, dt) = shapes[1]
    err, mism, n = compare_with_oracle(As[1], Bs[1], C2[1], M, N, K, dt)
    assert err <= TOL[dt]


# ---- split-K with the reduction fused into the GEMM launch (the k splits of a tile as one cluster) ----------

def fused_variants(M, N, K, dtype, lA=ROW, lB=ROW):
    return [(ab.adapt_matmul_plan_forced(M, N, K, dtype, lA, lB, c.tiling_key), c)
            for c in ab.adapt_plan_candidates(M, N, K, dtype, lA, lB) if c.fused]


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
@pytest.mark.parametrize("shape", [(1, 1024, 4096), (16, 512, 2048), (128, 384, 1024), (200, 264, 1328), (131, 77, 2590),
                                   (2048, 1024, 512), (8, 3001, 4000), (1030, 264, 1331), (300, 520, 390), (64, 64, 8192)])
def test_fused_split_k_bit_exact(shape, dtype):
    """Every fused configuration (cluster sizes 2, 4, 8; plain tiles, row-class tiles, k classes as the cluster's
    ranks; one tile per cluster and several) against the oracle on position-coded integers."""
    M, N, K = shape
    A = synth.position_coded(M, K, dtype, modulus=7, device="cuda")
    B = synth.position_coded(K, N, dtype, modulus=5, device="cuda").contiguous()
    variants = fused_variants(M, N, K, dtype)
    assert variants, "expected fused configurations for this shape"
    seen = set()
    for plan, c in variants:
        check_case(M, N, K, dtype, A, B, plan=plan, exact=True)
        seen.add(c.P_k)
    assert seen & {2, 4, 8}


@pytest.mark.parametrize("lA,lB", [(ROW, COL), (COL, ROW), (COL, COL)])
def test_fused_split_k_layouts(lA, lB):
    M, N, K = 136, 256, 2048
    for dtype in (ab.F16, ab.BF16):
        A = synth.position_coded(M, K, dtype, 7, "cuda")
        B = synth.position_coded(K, N, dtype, 5, "cuda")
        A_st = A.t().contiguous() if lA == COL else A
        B_st = B.t().contiguous() if lB == COL else B
        variants = fused_variants(M, N, K, dtype, lA, lB)
        assert variants
        for plan, c in variants:
            check_case(M, N, K, dtype, A_st, B_st, lA, lB, plan=plan, exact=True)


def test_fused_split_k_matches_the_two_launch_path_bit_for_bit_on_random_values():
    """Same split count, same ascending order of the additions: the fused reduction and the workspace reduction
    give the same bits, and the fused one is the same from run to run."""
    for (M, N, K, dtype) in [(16, 4096, 4096, ab.BF16), (128, 1024, 4096, ab.F16), (300, 200, 3000, ab.BF16)]:
        A = synth.draw_operand(M, K, synth.U11, 21, dtype, "cuda")
        B = synth.draw_operand(K, N, synth.U11, 22, dtype, "cuda")
        cands = ab.adapt_plan_candidates(M, N, K, dtype)
        for f in [c for c in cands if c.fused][:6]:
            twin = [c for c in cands if not c.fused and c.family == f.family and c.BN == f.BN and c.P_k == f.P_k
                    and c.srcA == f.srcA and c.srcB == f.srcB]
            pf = ab.adapt_matmul_plan_forced(M, N, K, dtype, ROW, ROW, f.tiling_key)
            C1 = run_library(A, B, M, N, K, dtype, plan=pf).clone()
            C2 = run_library(A, B, M, N, K, dtype, plan=pf)
            torch.cuda.synchronize()
            assert torch.equal(C1.view(torch.int16), C2.view(torch.int16))
            if twin:
                pt = ab.adapt_matmul_plan_forced(M, N, K, dtype, ROW, ROW, twin[0].tiling_key)
                C3 = run_library(A, B, M, N, K, dtype, plan=pt)
                torch.cuda.synchronize()
                assert torch.equal(C1.view(torch.int16), C3.view(torch.int16)), (f.BN, f.P_k)
            err, mism, n = compare_with_oracle(A, B, C1, M, N, K, dtype)
            assert err <= TOL[dtype]
        ab.adapt_poll_device_status(torch.cuda.current_stream().cuda_stream)


# ---- stream-K: the leftover wave's k-blocks shared by all slots, partials fixed up by the tile's owner ---------

def streamk_variants(M, N, K, dtype, lA=ROW, lB=ROW):
    return [(ab.adapt_matmul_plan_forced(M, N, K, dtype, lA, lB, c.tiling_key), c)
            for c in ab.adapt_plan_candidates(M, N, K, dtype, lA, lB) if c.streamk]


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
@pytest.mark.parametrize("shape", [(1000, 1024, 2048), (3000, 3000, 2048), (300, 520, 2100), (2560, 2048, 2048), (520, 520, 4096),
                                   (4096, 4096, 2048), (5000, 1000, 3000)])
def test_stream_k_bit_exact(shape, dtype):
    """Every stream-K configuration (1-CTA and pair tiles, fewer tiles than slots and several waves plus a
    leftover) against the oracle on position-coded integers, twice in a row on the same workspace."""
    M, N, K = shape
    A = synth.position_coded(M, K, dtype, modulus=7, device="cuda")
    B = synth.position_coded(K, N, dtype, modulus=5, device="cuda").contiguous()
    variants = streamk_variants(M, N, K, dtype)
    assert variants, "expected stream-K configurations for this shape"
    for plan, c in variants:
        check_case(M, N, K, dtype, A, B, plan=plan, exact=True)
        check_case(M, N, K, dtype, A, B, plan=plan, exact=True)


@pytest.mark.parametrize("lA,lB", [(ROW, COL), (COL, ROW), (COL, COL)])
def test_stream_k_layouts(lA, lB):
    M, N, K = 1160, 1000, 2048
    dtype = ab.BF16
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda")
    A_st = A.t().contiguous() if lA == COL else A
    B_st = B.t().contiguous() if lB == COL else B
    variants = streamk_variants(M, N, K, dtype, lA, lB)
    assert variants
    for plan, c in variants:
        check_case(M, N, K, dtype, A_st, B_st, lA, lB, plan=plan, exact=True)


def test_stream_k_random_values_run_twice_bit_identical():
    for (M, N, K, dtype) in [(4096, 4096, 4096, ab.F16), (3000, 3000, 3000, ab.BF16), (1000, 1024, 2048, ab.F16)]:
        A = synth.draw_operand(M, K, synth.U11, 31, dtype, "cuda")
        B = synth.draw_operand(K, N, synth.U11, 32, dtype, "cuda")
        for plan, c in streamk_variants(M, N, K, dtype)[:4]:
            C1 = run_library(A, B, M, N, K, dtype, plan=plan).clone()
            C2 = run_library(A, B, M, N, K, dtype, plan=plan)
            torch.cuda.synchronize()
            ab.adapt_poll_device_status(torch.cuda.current_stream().cuda_stream)
            assert torch.equal(C1.view(torch.int16), C2.view(torch.int16))
            rows = sample_rows(M, 48, seed=3)
            err, mism, n = compare_with_oracle(A, B, C1, M, N, K, dtype, rows=rows)
            assert err <= TOL[dtype], (c.BN, c.family, err)


# ---- row-class views on pair tiles (256 rows of one class per SM pair) ---------------------------------------

def pair_class_variants(M, N, K, dtype):
    return [(ab.adapt_matmul_plan_forced(M, N, K, dtype, ROW, ROW, c.tiling_key), c)
            for c in ab.adapt_plan_candidates(M, N, K, dtype) if c.srcA == 3 and c.family == ab.FAM_UMMA_2CTA]


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
@pytest.mark.parametrize("shape", [(131, 77, 259), (1030, 264, 331), (2500, 64, 1001), (16, 8, 9), (300, 520, 12), (2049, 128, 4099),
                                   (4100, 1000, 70), (5000, 16, 2047), (4096, 512, 1003)])
def test_pair_tiles_of_one_row_class_bit_exact(shape, dtype):
    """Both CTAs of a pair read 128 rows each of one row class of an A whose rows are not 16-byte aligned; every such
    configuration (TMA-store and thread-store epilogues, split-K) against the oracle on position-coded integers."""
    M, N, K = shape
    A = synth.position_coded(M, K, dtype, modulus=7, device="cuda")
    B = synth.position_coded(K, N, dtype, modulus=5, device="cuda")
    variants = pair_class_variants(M, N, K, dtype)
    assert variants, "shape must offer pair tiles of one row class"
    for plan, c in variants[:10]:
        check_case(M, N, K, dtype, A, B, plan=plan, exact=True)


def test_pair_tiles_of_one_row_class_do_not_leak_a_neighbouring_row():
    """As for the 1-CTA class tiles: non-finite values at the end of a row of A sit in front of the next row's
    first element in memory and must not reach that row's result, in either CTA of the pair."""
    M, N, K = 2600, 136, 203
    dtype = ab.F16
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda")
    bad_rows = [4, 17, 300, 1029, 1500, 2111]          # classes and halves of both CTAs
    for r in bad_rows:
        A[r, K - 1] = float("inf")
        A[r, K - 2] = float("nan")
    keep = torch.tensor([i for i in range(M) if i not in bad_rows], device="cuda")
    variants = pair_class_variants(M, N, K, dtype)
    assert variants
    for plan, c in variants[:6]:
        C = run_library(A, B, M, N, K, dtype, plan=plan)
        torch.cuda.synchronize()
        ab.adapt_poll_device_status(torch.cuda.current_stream().cuda_stream)
        assert torch.isfinite(C.index_select(0, keep)).all()
        err, mism, n = compare_with_oracle(A, B, C, M, N, K, dtype, rows=keep.cpu().numpy())
        assert mism == 0


def test_pair_tiles_of_one_row_class_random_values_and_unaligned_pointer():
    M, N, K, dtype = 3000, 688, 1999, ab.BF16
    A = synth.draw_operand(M, K, synth.U11, 81, dtype, "cuda")
    B = synth.draw_operand(K, N, synth.U11, 82, dtype, "cuda")
    bufA = torch.zeros(M * K + 8, dtype=torch.bfloat16, device="cuda")
    A1 = bufA[3:3 + M * K].view(M, K)
    A1.copy_(A)
    for plan, c in pair_class_variants(M, N, K, dtype)[:4]:
        for Ax in (A, A1):
            C = run_library(Ax, B, M, N, K, dtype, plan=plan)
            torch.cuda.synchronize()
            ab.adapt_poll_device_status(torch.cuda.current_stream().cuda_stream)
            rows = sample_rows(M, 64, seed=9)
            err, mism, n = compare_with_oracle(Ax, B, C, M, N, K, dtype, rows=rows)
            assert err <= TOL[dtype], (c.BN, c.P_k, err)


def test_shuffle_k_rotated_k_order_is_exact_and_reproducible():
    """ShuffleK: tiles walk their k-blocks in a rotated order.  Integer inputs stay bit-exact; random inputs stay within
    tolerance and give the same bits twice."""
    init()
    ab.adapt_set_option("shuffle_k", 1)
    try:
        for (M, N, K, dtype) in [(384, 512, 2048, ab.BF16), (1000, 1024, 1024, ab.F16), (2048, 2048, 512, ab.BF16)]:
            A = synth.position_coded(M, K, dtype, 7, "cuda")
            B = synth.position_coded(K, N, dtype, 5, "cuda")
            for plan, c in every_variant(M, N, K, dtype, families=(ab.FAM_UMMA_1CTA, ab.FAM_UMMA_2CTA), limit_per_family=6):
                check_case(M, N, K, dtype, A, B, plan=plan, exact=True)
            A = synth.draw_operand(M, K, synth.U11, 91, dtype, "cuda")
            B = synth.draw_operand(K, N, synth.U11, 92, dtype, "cuda")
            C1 = run_library(A, B, M, N, K, dtype).clone()
            C2 = run_library(A, B, M, N, K, dtype)
            torch.cuda.synchronize()
            assert torch.equal(C1.view(torch.int16), C2.view(torch.int16))
            err, mism, n = compare_with_oracle(A, B, C1, M, N, K, dtype)
            assert err <= TOL[dtype]
    finally:
        ab.adapt_set_option("shuffle_k", 0)
