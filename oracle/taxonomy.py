"""The paper's tiling taxonomy, data-volume and pipeline formulas -- TEST INFRASTRUCTURE ONLY.

Pure Python, written from the paper's definitions in its notation, used to pin
the host-side classifier and analytical model of the GPU library.  It shares no
code with that library.

Notation (Table 1): M, N, K input shape; m, n, k per-core sub-task; m1, n1, k1
on-chip tile; P_m = ceil(M/m), P_n = ceil(N/n), P_k = ceil(K/k); N_core cores;
S_L0C accumulator capacity in bytes (fp32 accumulation, 4 B per element).

Parity note: the absolute latency constants (lambda_r, eta_r, BW_r, Delta_dep
of Eq. 8-9) are hardware measurements the paper does not print, so absolute
predictions are "parity unpinned"; everything in this file is a closed form.
"""
from __future__ import annotations

from fractions import Fraction

COMMON = "Common"
SINGLE_CORE_SPLIT_K = "SingleCoreSplitK"
MULTI_CORE_SPLIT_K = "MultiCoreSplitK"
HYBRID_SPLIT_K = "HybridSplitK"


def ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def task_counts(M: int, N: int, K: int, m: int, n: int, k: int):
    """P_m, P_n, P_k of Table 1."""
    return ceil_div(M, m), ceil_div(N, n), ceil_div(K, k)


def accumulator_bytes(m1: int, n1: int) -> int:
    """Size of the fp32 accumulation tile, m1*n1*4 B (Section 4.1)."""
    return m1 * n1 * 4


def classify(M: int, N: int, m: int, n: int, m1: int, n1: int, N_core: int, S_L0C: int) -> str:
    """Section 4.2: the two axes of the template space.

    X axis, spatial parallelism: P_m * P_n >= N_core.
    Y axis, accumulation regime: m1 * n1 * 4 B <= S_L0C.
    """
    P_m, P_n = ceil_div(M, m), ceil_div(N, n)
    enough_tasks = P_m * P_n >= N_core
    fits_on_chip = accumulator_bytes(m1, n1) <= S_L0C
    if enough_tasks and fits_on_chip:
        return COMMON
    if enough_tasks and not fits_on_chip:
        return SINGLE_CORE_SPLIT_K
    if not enough_tasks and fits_on_chip:
        return MULTI_CORE_SPLIT_K
    return HYBRID_SPLIT_K


# ---- data volumes in bytes, 16-bit inputs and outputs, fp32 partial sums ----

def read_volume(M: int, N: int, K: int, m1: int, n1: int) -> Fraction:
    """Eq. 1: D_r = 2*M*N*K*(1/m1 + 1/n1)."""
    return 2 * M * N * K * (Fraction(1, m1) + Fraction(1, n1))


def write_volume_common(M: int, N: int) -> int:
    """Eq. 2: each output written once as 16 bits."""
    return 2 * M * N


def write_volume_single_core_split_k(M: int, N: int, K: int, k1: int) -> int:
    """Eq. 3: one fp32 spill per k1 slice plus the final 16-bit write."""
    return 4 * M * N * ceil_div(K, k1) + 2 * M * N


def write_volume_multi_core_split_k(M: int, N: int, K: int, k: int) -> int:
    """Eq. 4: one fp32 partial per K partition plus the final 16-bit write."""
    return 4 * M * N * ceil_div(K, k) + 2 * M * N


def write_volume_hybrid_split_k(M: int, N: int, K: int, k: int, k1: int) -> int:
    """Eq. 5, left-hand form: P_k partitions, each spilling once per k1 slice of its k range."""
    P_k = ceil_div(K, k)
    return P_k * (4 * M * N * ceil_div(k, k1)) + 2 * M * N


# ---- pipeline schedules for one tile of L slices (Eq. 12-14) ----------------

def t_baseline(L: int, t_M, t_P, T_drain):
    """Eq. 12: load and compute serialised across slices."""
    return L * (t_M + t_P) + T_drain


def t_double_buffer(L: int, t_M, t_P, T_drain):
    """Eq. 13: ping-pong buffers; a slice issues every max(t_M, t_P) after the fill."""
    return t_M + (L - 1) * max(t_M, t_P) + t_P + T_drain


def t_preload(Q: int, L: int, t_M, t_P, T_drain):
    """Eq. 14: Q tiles of L slices run as one continuous pipeline on a core."""
    return t_M + (Q * L - 1) * max(t_M, t_P) + t_P + Q * T_drain


def initiation_interval(stage_times, delta_dep=0):
    """Eq. 9: II = max over recurring stages + exposed dependency latency."""
    return max(stage_times) + delta_dep


def stage_cost(n_instr, lam, D_bytes, BW, eta):
    """Eq. 8: t = n*lambda + D / (BW * eta)."""
    return n_instr * lam + D_bytes / (BW * eta)


def main_loop(tiles):
    """Eq. 10: sum over a core's tiles of T_fill + (L-1)*II + T_drain.

    ``tiles`` is an iterable of (T_fill, L, II, T_drain).
    """
    return sum(T_fill + (L - 1) * II + T_drain for (T_fill, L, II, T_drain) in tiles)


def total_latency(T_pro, T_main_per_core, T_epi):
    """Eq. 7: prologue + slowest core's main loop + epilogue."""
    return T_pro + max(T_main_per_core) + T_epi
