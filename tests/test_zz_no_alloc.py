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
    before = torch.cuda.memory_allocated()
    for call in range(2):       # the scratch keeps the first call's partials: the second must still be right
        out = torch.full((M, N), float("nan"), dtype=A.dtype, device="cuda") if call == 0 else out.fill_(float("nan"))
        ab.adapt_matmul_noalloc(M, N, K, dtype, ab.ROW_MAJOR, ab.ROW_MAJOR, A.data_ptr(), B.data_ptr(), out.data_ptr(), stream)
        torch.cuda.synchronize()
        assert not torch.isnan(out).any()
        err = _rel_err(out, ref)
        # both results carry their own rounding to 16 bits, so allow twice the single-result bar
        assert err <= 2 * TOL[dtype], (call, err)
    assert torch.cuda.memory_allocated() - before <= out.numel() * 2 + 1024


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
