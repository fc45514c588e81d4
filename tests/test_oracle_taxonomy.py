"""Pins for the oracle's taxonomy / data-volume / pipeline formulas (no GPU)."""
import os
from fractions import Fraction

import pytest

from oracle import taxonomy as tx

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def worked_cases():
    out = []
    with open(os.path.join(GOLDEN, "taxonomy_cases.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            p = line.split()
            out.append(tuple(int(x) for x in p[:12]) + (p[12],))
    return out


@pytest.mark.parametrize("case", worked_cases())
def test_four_worked_cases_of_section_4_3(case):
    _, M, N, K, m, n, m1, n1, N_core, S, tasks, acc, template = case
    P_m, P_n, P_k = tx.task_counts(M, N, K, m, n, K)
    assert P_m * P_n == tasks and P_k == 1
    assert tx.accumulator_bytes(m1, n1) == acc
    assert tx.classify(M, N, m, n, m1, n1, N_core, S) == template


def test_case3_idle_cores():
    P_m, P_n, _ = tx.task_counts(128, 128, 4096, 64, 64, 4096)
    assert 16 - P_m * P_n == 12


def test_read_volume_eq1_from_first_principles():
    """Eq. 1 is the sum over tiles and slices of (m1*k1 + k1*n1) elements of 2 bytes."""
    M, N, K, m1, n1, k1 = 512, 768, 1024, 128, 256, 64
    tiles = (M // m1) * (N // n1)
    slices = K // k1
    by_count = 2 * tiles * slices * (m1 * k1 + k1 * n1)
    assert tx.read_volume(M, N, K, m1, n1) == by_count


def test_read_volume_case2_factor():
    """Growing 128x256 to 256x256 takes the factor (1/m1 + 1/n1) from 3/256 to 2/256."""
    a = tx.read_volume(4096, 4096, 1024, 128, 256)
    b = tx.read_volume(4096, 4096, 1024, 256, 256)
    unit = 2 * 4096 * 4096 * 1024
    assert a / unit == Fraction(3, 256) and b / unit == Fraction(2, 256)
    assert b / a == Fraction(2, 3)


def test_write_volumes_eq2_to_eq5():
    M, N, K = 300, 500, 4096
    assert tx.write_volume_common(M, N) == 2 * M * N
    assert tx.write_volume_single_core_split_k(M, N, K, 512) == 4 * M * N * 8 + 2 * M * N
    assert tx.write_volume_multi_core_split_k(M, N, K, 1024) == 4 * M * N * 4 + 2 * M * N
    # no split (k = K) leaves one fp32 partial plus the final write
    assert tx.write_volume_multi_core_split_k(M, N, K, K) == 6 * M * N
    # Eq. 5: when k1 | k and k | K the hybrid volume equals the single-core one
    assert (tx.write_volume_hybrid_split_k(M, N, K, 1024, 256)
            == tx.write_volume_single_core_split_k(M, N, K, 256))
    # ... and exceeds it when the divisibility fails (ceil taken per partition)
    assert (tx.write_volume_hybrid_split_k(M, N, 4000, 1000, 300)
            > tx.write_volume_single_core_split_k(M, N, 4000, 300))


def test_classifier_monotone_in_M_and_N():
    for M in range(64, 4096, 331):
        for N in range(64, 4096, 517):
            c = tx.classify(M, N, 128, 128, 128, 128, 148, 256 * 1024)
            if c == tx.COMMON:
                assert tx.classify(M + 128, N, 128, 128, 128, 128, 148, 256 * 1024) == tx.COMMON
                assert tx.classify(M, N + 128, 128, 128, 128, 128, 148, 256 * 1024) == tx.COMMON


@pytest.mark.parametrize("L", [1, 2, 7, 64])
@pytest.mark.parametrize("tM,tP", [(3, 5), (5, 3), (4, 4), (Fraction(1, 3), 2)])
def test_pipeline_identities_eq12_to_eq14(L, tM, tP):
    D = 7
    base = tx.t_baseline(L, tM, tP, D)
    db = tx.t_double_buffer(L, tM, tP, D)
    assert db <= base
    assert base - db == (L - 1) * min(tM, tP)
    for Q in (1, 3, 10):
        pre = tx.t_preload(Q, L, tM, tP, D)
        assert Q * db - pre == (Q - 1) * min(tM, tP)
    if L == 1:
        assert base == db == tx.t_preload(1, 1, tM, tP, D) == tM + tP + D


def test_pipeline_by_event_simulation():
    """Eq. 13 from a direct simulation of a two-buffer load/compute pipeline."""
    for L in (1, 2, 5, 9):
        for tM, tP in ((3, 5), (5, 3), (2, 2)):
            load_done = [0] * L
            comp_done = [0] * L
            for s in range(L):
                # a buffer is free once the slice two steps back has been consumed
                start_load = max(load_done[s - 1] if s else 0, comp_done[s - 2] if s >= 2 else 0)
                load_done[s] = start_load + tM
                start_comp = max(load_done[s], comp_done[s - 1] if s else 0)
                comp_done[s] = start_comp + tP
            assert comp_done[-1] == tx.t_double_buffer(L, tM, tP, 0)


def test_main_loop_and_total_eq7_eq10():
    tiles = [(2, 10, 3, 1), (2, 1, 3, 1)]
    assert tx.main_loop(tiles) == (2 + 9 * 3 + 1) + (2 + 0 + 1)
    assert tx.total_latency(5, [10, 30, 20], 7) == 42
    assert tx.initiation_interval([3, 9, 4], 2) == 11
    assert tx.stage_cost(4, 10, 1000, 100, Fraction(1, 2)) == 40 + 20
