"""GPU parity of the operators beside MatMul (Section 6.5: AddMM, BatchMM, GroupMM) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import gemm as og
from paper_2608_10803_b200 import binding as ab
from paper_2608_10803_b200 import synth

from gpu_util import TOL, init, sample_rows

pytestmark = pytest.mark.gpu


def run_addmm(M, N, K, dtype, A, B, D, alpha, beta, plan=None, out=None):
    init()
    st = torch.cuda.current_stream().cuda_stream
    if plan is None:
        plan = ab.adapt_matmul_plan(M, N, K, dtype)
    if out is None:
        out = torch.full((M, N), float("nan"), dtype=A.dtype, device="cuda")
    ab.adapt_addmm(plan, A.data_ptr(), B.data_ptr(), D.data_ptr(), D.numel() == N and M * N != N, alpha, beta, out.data_ptr(), st)
    torch.cuda.synchronize()
    ab.adapt_poll_device_status(st)
    return out


def variants(M, N, K, dtype, limit=3):
    """A few forced plans of every family (AddMM must work whatever the plan's kernel is)."""
    out, seen = [None], {}
    for c in ab.adapt_plan_candidates(M, N, K, dtype):
        key = (c.family, c.srcA, c.srcB, c.P_k > 1, c.fused, c.streamk)
        if seen.get(key, 0) >= 1 or len(out) > 24:
            continue
        seen[key] = 1
        out.append(ab.adapt_matmul_plan_forced(M, N, K, dtype, 0, 0, c.tiling_key))
    return out


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
@pytest.mark.parametrize("shape", [(256, 256, 256), (131, 77, 259), (1000, 1024, 1024), (5, 640, 1000), (300, 520, 12), (64, 64, 8192),
                                   (1030, 265, 331), (8, 3001, 400)])
def test_addmm_integers_bit_exact_matrix_and_bias(shape, dtype):
    M, N, K = shape
    A = synth.position_coded(M, K, dtype, 7, "cuda")
    B = synth.position_coded(K, N, dtype, 5, "cuda").contiguous()
    Dm = synth.draw_operand(M, N, ("integer", -8, 8), 41, dtype, "cuda")
    Dv = synth.draw_operand(1, N, ("integer", -8, 8), 42, dtype, "cuda").reshape(-1)
    for plan in variants(M, N, K, dtype):
        for D, alpha, beta in ((Dm, 1.0, 1.0), (Dv, 2.0, -3.0), (Dm, -1.0, 0.5)):
            C = run_addmm(M, N, K, dtype, A, B, D, alpha, beta, plan=plan)
            _, O16 = og.addmm_rows(synth.bits(A), synth.bits(B), synth.bits(D), M, N, K, dtype, alpha, beta)
            mism = int(np.count_nonzero(synth.bits(C).reshape(O16.shape) != O16))
            assert mism == 0, (shape, dtype, alpha, beta, mism)


@pytest.mark.parametrize("dtype", [ab.F16, ab.BF16])
def test_addmm_random_values_within_tolerance_and_in_place(dtype):
    for (M, N, K) in [(2048, 1024, 512), (333, 4100, 777), (16, 4096, 4096)]:
        A = synth.draw_operand(M, K, synth.U11, 51, dtype, "cuda")
        B = synth.draw_operand(K, N, synth.U11, 52, dtype, "cuda")
        D = synth.draw_operand(M, N, synth.U11, 53, dtype, "cuda")
        alpha, beta = 0.3, -1.7
        C = run_addmm(M, N, K, dtype, A, B, D, alpha, beta)
        rows = sample_rows(M, 64, seed=5)
        O64, _ = og.addmm_rows(synth.bits(A), synth.bits(B), synth.bits(D), M, N, K, dtype, alpha, beta, rows=rows)
        idx = torch.from_numpy(rows).cuda()
        err, bad = og.rel_fro_error(synth.bits(C.index_select(0, idx)), O64, dtype)
        assert bad == 0 and err <= TOL[dtype], (M, N, K, err)
        # in place: C = beta * C + alpha * A * B gives the same bits
        Cin = D.clone()
        run_addmm(M, N, K, dtype, A, B, Cin, alpha, beta, out=Cin)
        assert torch.equal(Cin.view(torch.int16), C.view(torch.int16))


def test_addmm_degenerate_and_errors():
    init()
    st = torch.cuda.current_stream().cuda_stream
    dtype = ab.F16
    D = synth.draw_operand(4, 6, ("integer", -8, 8), 61, dtype, "cuda")
    C = torch.full((4, 6), float("nan"), dtype=torch.float16, device="cuda")
    A = torch.ones((4, 1), dtype=torch.float16, device="cuda")
    plan = ab.adapt_matmul_plan(4, 6, 0, dtype)                 # K == 0: beta * D
    ab.adapt_addmm(plan, A.data_ptr(), A.data_ptr(), D.data_ptr(), False, 1.0, 2.0, C.data_ptr(), st)
    torch.cuda.synchronize()
    assert torch.equal(C, 2 * D)
    plan = ab.adapt_matmul_plan(64, 64, 64, dtype)
    X = torch.ones((64, 64), dtype=torch.float16, device="cuda")
    Y = torch.ones((64, 64), dtype=torch.float16, device="cuda")
    with pytest.raises(ab.AdaptError) as e:
        ab.adapt_addmm(plan, X.data_ptr(), Y.data_ptr(), Y.data_ptr() + 2, False, 1.0, 1.0, Y.data_ptr(), st)   # D overlaps C, is not C
    assert e.value.status == ab.ERR_INVALID_ARG
    with pytest.raises(ab.AdaptError) as e:
        ab.adapt_addmm(plan, X.data_ptr(), Y.data_ptr(), 0, False, 1.0, 1.0, X.data_ptr(), st)
    assert e.value.status == ab.ERR_INVALID_ARG


def test_strided_batch_matches_the_oracle_per_entry():
    init()
    st = torch.cuda.current_stream().cuda_stream
    for (M, N, K, dtype, batch) in [(131, 77, 259, ab.BF16, 5), (256, 512, 1024, ab.F16, 3), (8, 3001, 400, ab.F16, 2)]:
        A = synth.draw_operand(batch * M, K, ("integer", -4, 4), 71, dtype, "cuda")
        B = synth.draw_operand(K, N, ("integer", -4, 4), 72, dtype, "cuda")           # shared by the batch: stride 0
        C = torch.full((batch * M, N), float("nan"), dtype=A.dtype, device="cuda")
        plan = ab.adapt_matmul_plan(M, N, K, dtype)
        ab.adapt_matmul_strided_batch(plan, A.data_ptr(), M * K, B.data_ptr(), 0, C.data_ptr(), M * N, batch, st)
        torch.cuda.synchronize()
        ab.adapt_poll_device_status(st)
        for b in range(batch):
            _, C16 = og.gemm(synth.bits(A[b * M:(b + 1) * M]), synth.bits(B), M, N, K, dtype)
            assert np.array_equal(synth.bits(C[b * M:(b + 1) * M]).reshape(C16.shape), C16), (M, N, K, b)
    with pytest.raises(ab.AdaptError):
        ab.adapt_matmul_strided_batch(plan, A.data_ptr(), M * K, B.data_ptr(), 0, C.data_ptr(), M * N - 1, 2, st)
