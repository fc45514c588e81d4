"""Helpers for the GPU parity tests: run the library through its C ABI on seeded inputs and
compare with the CPU oracle (full output, or complete sampled rows for large shapes)."""
from __future__ import annotations

import numpy as np
import torch

from oracle import gemm as og
from paper_2608_10803_b200 import binding as ab
from paper_2608_10803_b200 import synth

TOL = {ab.F16: 1e-3, ab.BF16: 8e-3}     # normwise ||C - C_ref||_F / ||C_ref||_F, norms in fp64

def init():
    ab.adapt_init(0)        # idempotent, and a test elsewhere may have shut the library down


def run_library(A: torch.Tensor, B: torch.Tensor, M: int, N: int, K: int, dtype: int,
                layoutA=ab.ROW_MAJOR, layoutB=ab.ROW_MAJOR, plan=None, out=None) -> torch.Tensor:
    """C (M x N, row-major, device) = A * B through adapt_matmul on the current stream."""
    init()
    if plan is None:
        plan = ab.adapt_matmul_plan(M, N, K, dtype, layoutA, layoutB)
    if out is None:
        out = torch.full((M, N), float("nan"), dtype=synth.torch_dtype(dtype), device="cuda")
    ab.adapt_matmul(plan, A.data_ptr() if A.numel() else 0, B.data_ptr() if B.numel() else 0,
                    out.data_ptr() if out.numel() else 0, torch.cuda.current_stream().cuda_stream)
    return out


def sample_rows(M: int, count: int, seed: int = 0) -> np.ndarray:
    """Complete output rows to check: the corners, one row per residue class region of the
    128-row tile, and seeded random rows."""
    if M <= count:
        return np.arange(M, dtype=np.int64)
    rng = np.random.default_rng(seed)
    fixed = [0, 1, M - 1, M - 2, 127 % M, 128 % M, 129 % M, 255 % M, 256 % M, (M // 2) % M, (M // 2 + 63) % M]
    rest = rng.choice(M, max(0, count - len(fixed)), replace=False).tolist()
    return np.array(sorted(set(fixed + rest)), dtype=np.int64)


def rows_for_budget(M: int, N: int, K: int, mac_budget: float = 4e9, min_rows: int = 24, max_rows: int = 512) -> int:
    per_row = max(1, N * K)
    return int(max(min_rows, min(max_rows, mac_budget // per_row)))


def compare_with_oracle(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor, M, N, K, dtype,
                        layoutA=ab.ROW_MAJOR, layoutB=ab.ROW_MAJOR, rows=None):
    """Returns (relative Frobenius error over the checked rows, number of 16-bit mismatches
    against the oracle's directly rounded result, number of elements checked)."""
    A_bits = synth.bits(A).reshape(-1)
    B_bits = synth.bits(B).reshape(-1)
    if rows is None:
        C64, C16 = og.gemm(A_bits, B_bits, M, N, K, dtype, layoutA, layoutB)
        got = synth.bits(C)
    else:
        rows = np.asarray(rows, dtype=np.int64)
        C64, C16 = og.gemm_rows(A_bits, B_bits, M, N, K, dtype, layoutA, layoutB, rows=rows)
        idx = torch.from_numpy(rows).to(C.device)
        got = synth.bits(C.index_select(0, idx))
    err, bad = og.rel_fro_error(got, C64, dtype)
    assert bad == 0, f"{bad} non-finite differences"
    mism = int(np.count_nonzero(got.reshape(C16.shape) != C16))
    return err, mism, int(C16.size)


def check_case(M, N, K, dtype, A, B, layoutA=ab.ROW_MAJOR, layoutB=ab.ROW_MAJOR, plan=None,
               mac_budget=4e9, exact=False, seed=0):
    """Run one GEMM and assert the acceptance bar; returns (err, mismatches, checked, info)."""
    C = run_library(A, B, M, N, K, dtype, layoutA, layoutB, plan)
    torch.cuda.synchronize()
    ab.adapt_poll_device_status(torch.cuda.current_stream().cuda_stream)
    rows = None
    if M * N * K > mac_budget:
        rows = sample_rows(M, rows_for_budget(M, N, K, mac_budget), seed)
    err, mism, n = compare_with_oracle(A, B, C, M, N, K, dtype, layoutA, layoutB, rows)
    h = plan if plan is not None else ab.adapt_matmul_plan(M, N, K, dtype, layoutA, layoutB)
    info = ab.adapt_plan_info(h)
    tag = f"{M}x{N}x{K} dt{dtype} {ab.FAMILY_NAMES[info.family]} {info.BM}x{info.BN} st{info.stages} P_k{info.P_k}"
    if exact:
        assert mism == 0, f"{tag}: {mism}/{n} elements differ from the exact result"
    assert err <= TOL[dtype], f"{tag}: relative error {err:.3e} above {TOL[dtype]:.0e}"
    return err, mism, n, info
