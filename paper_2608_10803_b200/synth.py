"""Seeded synthetic inputs: shapes and operand values.

This module holds no GEMM arithmetic.  It only draws shapes and 16-bit operand
values (fp32 draw, one round-to-nearest-even cast to fp16/bf16 by torch) and is
the one module both the CPU oracle's tests and the GPU harness may use, so that
both sides see the same bits.

Workloads (stand-ins for the paper's private ~80,000-shape industrial set and
its recommendation-model layers, Section 6.1):

* ``CONFIG_SQUARE``   single 256^3 fp16 GEMM, U[-1,1], seed 0
* ``config_reco()``   N=K=1024, M in {1,7,64,1000,10000,100000}, fp16
* ``config_llm()``    M in {1,16,128,2048,8192} x four (N,K) layer shapes, bf16
* ``config_large()``  8192^3, 16384x16384x4096, 256x256x262144, bf16
* ``sweep_shapes()``  2,000 shapes, M,N,K log-uniform in [1,1e5], M*N*K <= 2^38
"""
from __future__ import annotations

import csv
import os
from dataclasses import dataclass

import numpy as np
import torch

F16 = 0
BF16 = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
SWEEP_CSV = os.path.join(_HERE, "data", "sweep_shapes.csv")


@dataclass(frozen=True)
class GemmCase:
    """One GEMM problem of a workload: shape, dtype and how its operands are drawn."""
    config: int
    index: int
    M: int
    N: int
    K: int
    dtype: int            # F16 or BF16
    distA: tuple          # ("uniform", lo, hi) or ("normal", mean, std)
    distB: tuple
    seedA: int
    seedB: int

    @property
    def name(self) -> str:
        return f"c{self.config}_{self.M}x{self.N}x{self.K}_{'bf16' if self.dtype else 'f16'}"

    @property
    def flops(self) -> float:
        return 2.0 * self.M * self.N * self.K

    @property
    def bytes(self) -> float:
        return 2.0 * (self.M * self.K + self.K * self.N + self.M * self.N)


def _seeds(config: int, index: int):
    base = 1_000_003 * config + 2 * index
    return base, base + 1


def _case(config, index, M, N, K, dtype, distA, distB, seeds=None):
    sA, sB = seeds if seeds else _seeds(config, index)
    return GemmCase(config, index, int(M), int(N), int(K), dtype, distA, distB, sA, sB)


U11 = ("uniform", -1.0, 1.0)


def config_square():
    return [_case(1, 0, 256, 256, 256, F16, U11, U11, seeds=(0, 1))]


def config_reco():
    K = 1024
    distB = ("normal", 0.0, 1.0 / np.sqrt(K))
    return [_case(2, i, M, 1024, K, F16, U11, distB)
            for i, M in enumerate([1, 7, 64, 1000, 10000, 100000])]


LLM_NK = [(4096, 4096), (14336, 4096), (4096, 14336), (128256, 4096)]
LLM_M = [1, 16, 128, 2048, 8192]


def config_llm():
    out = []
    i = 0
    for (N, K) in LLM_NK:
        for M in LLM_M:
            out.append(_case(3, i, M, N, K, BF16, ("normal", 0.0, 1.0), ("normal", 0.0, 0.02)))
            i += 1
    return out


def config_large():
    shapes = [(8192, 8192, 8192), (16384, 16384, 4096), (256, 256, 262144)]
    return [_case(4, i, M, N, K, BF16, U11, U11) for i, (M, N, K) in enumerate(shapes)]


def draw_sweep_shapes(count: int = 2000, seed: int = 42, limit: int = 2 ** 38):
    """The sweep recipe itself: log-uniform dims in [1, 1e5], rejection on M*N*K <= limit."""
    rng = np.random.default_rng(seed)
    shapes = []
    draws = 0
    while len(shapes) < count:
        u = rng.random(3)
        draws += 1
        m, n, k = (int(v) for v in np.clip(np.floor(np.exp(u * np.log(100000.0))), 1, 100000))
        if m * n * k <= limit:
            shapes.append((m, n, k))
    return shapes, draws


def sweep_shapes():
    """The 2,000 (M, N, K) triples, read from the committed CSV (written by ``data/make_sweep.py``)."""
    with open(SWEEP_CSV, newline="") as f:
        rd = csv.reader(f)
        header = next(rd)
        assert header == ["index", "M", "N", "K"], header
        return [(int(r[1]), int(r[2]), int(r[3])) for r in rd]


def config_sweep():
    return [_case(5, i, M, N, K, F16 if i % 2 == 0 else BF16, U11, U11)
            for i, (M, N, K) in enumerate(sweep_shapes())]


def sweep_like(seed: int, count: int):
    """A second shape set drawn with the sweep's recipe from another seed (held-out shapes for the model check)."""
    shapes, _ = draw_sweep_shapes(count, seed)
    return [_case(7, i, M, N, K, F16 if i % 2 == 0 else BF16, U11, U11) for i, (M, N, K) in enumerate(shapes)]


def sweep_oracle_subset(count: int = 200, seed: int = 43, total: int = 2000):
    """Indices of the sweep shapes that are checked against the oracle."""
    return sorted(int(i) for i in np.random.default_rng(seed).choice(total, count, replace=False))


def config_context():
    """Shapes the paper names in its text (Sections 2.2, 6.3, 6.4); fp16, U[-1,1]."""
    shapes = [(12288, 688, 16991), (3, 256, 87087), (4096, 4096, 4096), (256, 65536, 4096)]
    return [_case(6, i, M, N, K, F16, U11, U11) for i, (M, N, K) in enumerate(shapes)]


# ---- operand values ---------------------------------------------------------

def torch_dtype(dtype: int):
    return torch.float16 if dtype == F16 else torch.bfloat16


def draw_operand(rows: int, cols: int, dist: tuple, seed: int, dtype: int, device="cpu") -> torch.Tensor:
    """A rows x cols operand: fp32 draw from ``dist`` with ``seed``, one RN-even cast to 16 bits."""
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    n = rows * cols
    out = torch.empty(n, dtype=torch_dtype(dtype), device=device)
    # draw in chunks so a multi-GB operand never needs an fp32 copy of itself
    chunk = 1 << 26
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        if dist[0] == "uniform":
            x = torch.rand(hi - lo, generator=g, device=device, dtype=torch.float32)
            x = x * (dist[2] - dist[1]) + dist[1]
        elif dist[0] == "normal":
            x = torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32)
            x = x * dist[2] + dist[1]
        elif dist[0] == "integer":
            x = torch.randint(int(dist[1]), int(dist[2]) + 1, (hi - lo,), generator=g, device=device).float()
        else:
            raise ValueError(dist)
        out[lo:hi] = x.to(out.dtype)
    return out.view(rows, cols)


def draw_case(case: GemmCase, device="cpu"):
    """(A [M,K], B [K,N]) row-major for one workload case."""
    A = draw_operand(case.M, case.K, case.distA, case.seedA, case.dtype, device)
    B = draw_operand(case.K, case.N, case.distB, case.seedB, case.dtype, device)
    return A, B


def bits(t: torch.Tensor) -> np.ndarray:
    """Raw 16-bit words of an fp16/bf16 tensor as a host uint16 array."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def from_bits(b: np.ndarray, dtype: int, device="cpu") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).to(device).view(torch_dtype(dtype))


def position_coded(rows: int, cols: int, dtype: int, modulus: int = 7, device="cpu") -> torch.Tensor:
    """Small-integer matrix whose entry depends on its own (row, col): a mis-addressed element shows."""
    r = torch.arange(rows, device=device).view(-1, 1)
    c = torch.arange(cols, device=device).view(1, -1)
    v = ((r * 3 + c * 5 + (r * c) % 11) % modulus) - (modulus // 2)
    return v.to(torch_dtype(dtype))
