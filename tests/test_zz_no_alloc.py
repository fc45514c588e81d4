"""The allocation-free entry point (adapt_matmul_noalloc), checked against the regular one.

Some callers cannot allocate device memory: a serving loop that must never hit the implicit
synchronisation of cudaMalloc, a process that gave all device memory to another allocator, a
plug-in that only receives buffers and a stream.  For them the library keeps a fixed 4 MiB
scratch inside its own image and offers one call that uses it.  This file is collected last on
purpose, so that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import gemm as og
from paper_2608_10803_b200 import binding as ab
from paper_2608_10803_b200 import synth

pytestmark = pytest.mark.gpu

TOL = {ab.F16: 1e-3, ab.BF16: 8e-3}


def _rel_err(got: torch.Tensor, ref: torch.Tensor) -> float:
    g, r = got.double(), ref.double()
    return float(torch.linalg.norm(g - r) / torch.linalg.norm(r))


@pytest.mark.parametrize("shape,dtype", [((300, 520, 4100), ab.F16), ((131, 77, 2590), ab.BF16), ((64, 1000, 777), ab.F16)])
def test_noalloc_matches_regular_entry_point_twice_in_a_row(shape, dtype):
    M, N, K = shape
    ab.adapt_init(0)            # only the regular entry point needs it
    stream = torch.cuda.current_stream().cuda_stream
    A = synth.draw_operand(M, K, synth.U11, 11, dtype, "cuda")
    B = synth.draw_operand(K, N, synth.U11, 12, dtype, "cuda")
    ref = torch.empty((M, N), dtype=A.dtype, device="cuda")
    ab.adapt_matmul(ab.adapt_matmul_plan(M, N, K, dtype), A.data_ptr(), B.data_ptr(), ref.data_ptr(), stream)
    torch.cuda.synchronize()
    out = torch.full((M, N), float("nan"), dtype=A.dtype, device="cuda")
    ab.adapt_matmul_noalloc(M, N, K, dtype, ab.ROW_MAJOR, ab.ROW_MAJOR, A.data_ptr(), B.data_ptr(), out.data_ptr(), stream)
    torch.cuda.synchronize()    # the first call on a device looks up the scratch address; from here on nothing may be allocated
    assert not torch.isnan(out).any() and _rel_err(out, ref) <= 2 * TOL[dtype]   # also fills torch's own block cache for the checks below
    free_before = torch.cuda.mem_get_info()[0]      # the driver's own figure: sees every cudaMalloc, not just torch's
    for call in range(2):       # the scratch keeps the first call's partials: the second must still be right
        out.fill_(float("nan"))
        ab.adapt_matmul_noalloc(M, N, K, dtype, ab.ROW_MAJOR, ab.ROW_MAJOR, A.data_ptr(), B.data_ptr(), out.data_ptr(), stream)
        torch.cuda.synchronize()
        assert not torch.isnan(out).any()
        err = _rel_err(out, ref)
        # both results carry their own rounding to 16 bits, so allow twice the single-result bar
        assert err <= 2 * TOL[dtype], (call, err)
    # torch allocates nothing between the two readings either (out is reused), so the device's free memory
    # may only move by what other processes on a shared GPU do: allow a small slack
    assert free_before - torch.cuda.mem_get_info()[0] <= (2 << 20)
    # and against the oracle itself, not only against the regular entry point
    rows = np.arange(0, M, max(1, M // 24), dtype=np.int64)
    C64, _ = og.gemm_rows(synth.bits(A).reshape(-1), synth.bits(B).reshape(-1), M, N, K, dtype, rows=rows)
    err, bad = og.rel_fro_error(synth.bits(out.index_select(0, torch.from_numpy(rows).cuda())), C64, dtype)
    assert bad == 0 and err <= TOL[dtype], err


def test_noalloc_exact_on_integers_and_after_a_different_shape():
    """Small integers: bit-identical to the regular path, also right after a call with another shape
    left other partials in the scratch."""
    stream = torch.cuda.current_stream().cuda_stream
    ab.adapt_init(0)
    for (M, N, K) in [(200, 264, 328), (57, 33, 1000), (200, 264, 328)]:
        A = synth.position_coded(M, K, ab.F16, 7, "cuda")
        B = synth.position_coded(K, N, ab.F16, 5, "cuda")
        ref = torch.empty((M, N), dtype=torch.float16, device="cuda")
        out = torch.empty_like(ref)
        ab.adapt_matmul(ab.adapt_matmul_plan(M, N, K, ab.F16), A.data_ptr(), B.data_ptr(), ref.data_ptr(), stream)
        ab.adapt_matmul_noalloc(M, N, K, ab.F16, 0, 0, A.data_ptr(), B.data_ptr(), out.data_ptr(), stream)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))


def test_noalloc_rejects_outputs_beyond_the_scratch():
    A = torch.zeros(8, dtype=torch.float16, device="cuda")
    with pytest.raises(ab.AdaptError) as e:
        ab.adapt_matmul_noalloc(2048, 2048, 64, ab.F16, 0, 0, A.data_ptr(), A.data_ptr(), A.data_ptr(), 0)
    assert e.value.status == ab.ERR_UNSUPPORTED and "4 MiB" in str(e.value)
    with pytest.raises(ab.AdaptError) as e:
        ab.adapt_matmul_noalloc(0, 4, 4, ab.F16, 0, 0, A.data_ptr(), A.data_ptr(), A.data_ptr(), 0)
    assert e.value.status == ab.ERR_INVALID_ARG


def test_noalloc_needs_neither_init_nor_a_plan():
    """In a fresh process that never calls adapt_init or makes a plan, the entry point alone gives the
    oracle's result (bit-exact on small integers)."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = r"""
import sys
sys.path.insert(0, %r)
import numpy as np, torch
from oracle import gemm as og
from paper_2608_10803_b200 import binding as ab, synth
M, N, K, dt = 190, 203, 777, ab.BF16
A = synth.position_coded(M, K, dt, 7, "cuda")
B = synth.position_coded(K, N, dt, 5, "cuda")
C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
for _ in range(2):
    ab.adapt_matmul_noalloc(M, N, K, dt, 0, 0, A.data_ptr(), B.data_ptr(), C.data_ptr(), torch.cuda.current_stream().cuda_stream)
torch.cuda.synchronize()
_, C16 = og.gemm(synth.bits(A).reshape(-1), synth.bits(B).reshape(-1), M, N, K, dt)
assert np.array_equal(synth.bits(C).reshape(C16.shape), C16)
assert ab.adapt_plan_cache_size() == 0
print("NOALLOC_OK")
""" % root
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "NOALLOC_OK" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
