"""Pins of the oracle's batch-size controller (Eq. 6-8, getBsz, evalBsz) against hand-derived
traces, the closed form b* = T * tbar, brute force over the shift of Eq. 8, and invariants."""
import itertools
import json
from pathlib import Path

import numpy as np
import pytest

from oracle import oracle as O

GOLD = json.loads((Path(__file__).parent / "golden" / "controller_cases.json").read_text())


@pytest.mark.parametrize("case", GOLD["cases"], ids=lambda c: c["name"].split()[0])
def test_hand_derived_traces(case):
    mode = O.MODE_BSP if case["mode"] == "bsp" else O.MODE_ASP
    c = O.Controller(case["K"], case["B"], case["b_min"], case["b_max"], case["deadband"], 1.0, mode)
    assert c.batches.tolist() == case["b0"]          # Alg. 1: b = B / K
    for want in case["expect"]:
        nb, ch = c.rebatch(case["throughput"])
        assert nb.tolist() == want
        assert c.batches.tolist() == want


def test_bstar_is_throughput_times_mean_time():
    """Eq. 6b collapses: b - (b/t)(t - tbar) = (b/t) tbar = T tbar."""
    rng = np.random.default_rng(1)
    for _ in range(200):
        K = int(rng.integers(1, 33))
        b0 = rng.integers(1, 200, K).astype(np.int32)
        T = rng.uniform(0.1, 50.0, K)
        c = O.Controller(K, int(b0.sum()), 1, 100000, 0.0, 1.0, O.MODE_ASP)
        c.set_batches(b0)
        _, _, bstar = c.rebatch(T, want_bstar=True)
        tbar = np.mean(b0 / T)
        np.testing.assert_allclose(bstar, T * tbar, rtol=1e-12)


def test_equal_batches_grow_the_global_batch_by_am_hm():
    """With equal b the sum of b* is B * mean(T) * mean(1/T) >= B (the growth Eq. 8 removes)."""
    rng = np.random.default_rng(2)
    for _ in range(50):
        K = int(rng.integers(2, 17))
        T = rng.uniform(1.0, 8.0, K)
        c = O.Controller(K, 32 * K, 1, 100000, 0.0, 1.0, O.MODE_ASP)
        _, _, bstar = c.rebatch(T, want_bstar=True)
        want = 32 * K * T.mean() * (1.0 / T).mean()
        assert abs(bstar.sum() - want) <= 1e-10 * want
        assert bstar.sum() >= 32 * K * (1 - 1e-12)


def _shift_by_search(n_pre, B, b_min, b_max):
    """Eq. 8 restated without a loop over units: find the number s of whole rounds such that
    clamping n_pre -/+ s leaves fewer units than there are movable workers, then hand the rest
    to the largest movable batches (lowest index first among equals)."""
    n_pre = list(n_pre)
    D = B - sum(n_pre)
    if D == 0:
        return n_pre
    d = 1 if D > 0 else -1
    for s in range(0, 100000):
        base = [min(b_max, x + s) if d > 0 else max(b_min, x - s) for x in n_pre]
        rest = (B - sum(base)) * d
        movable = [k for k, x in enumerate(base) if (x < b_max if d > 0 else x > b_min)]
        if 0 <= rest < max(len(movable), 1) or (rest == 0):
            order = sorted(movable, key=lambda k: (-base[k], k))[:rest]
            for k in order:
                base[k] += d
            return base
    raise AssertionError("no shift found")


def test_conservation_matches_search_over_the_shift():
    """Wide dead-band off, so the pre-conservation integers are floor(T tbar + 1/2), clamped."""
    rng = np.random.default_rng(3)
    for _ in range(400):
        K = int(rng.integers(2, 9))
        per = int(rng.integers(4, 40))
        B = K * per
        b_min = int(rng.integers(1, max(2, per // 2)))
        b_max = int(rng.integers(per + 1, 4 * per))
        T = rng.uniform(1.0, 8.0, K)
        c = O.Controller(K, B, b_min, b_max, 0.0, 1.0, O.MODE_BSP)
        tbar = np.mean(per / T)
        n_pre = np.clip(np.floor(np.clip(T * tbar, b_min, b_max) + 0.5), b_min, b_max).astype(int)
        nb, _ = c.rebatch(T)
        assert nb.tolist() == _shift_by_search(n_pre, B, b_min, b_max)


def test_exhaustive_small_invariants():
    """Sum b = B and bounds after every synchronous re-batch, for every throughput pattern on a
    small grid and several consecutive re-batches."""
    levels = (1.0, 2.0, 3.0, 8.0)
    for K in (2, 3, 4):
        for B in (K * 4, K * 5 + 1, K * 16):
            for T in itertools.product(levels, repeat=K):
                c = O.Controller(K, B, 2, 3 * (B // K), 0.1, 1.0, O.MODE_BSP)
                assert c.batches.sum() == B and c.batches.max() - c.batches.min() <= 1
                for _ in range(4):
                    nb, ch = c.rebatch(T)
                    assert nb.sum() == B
                    assert nb.min() >= 2 and nb.max() <= 3 * (B // K)


def test_fixed_point_when_throughput_proportional_to_batch():
    """t_k all equal => every error is zero => nothing changes, for any dead-band including 0."""
    for db in (0.0, 0.1):
        c = O.Controller(4, 64, 2, 48, db, 1.0, O.MODE_BSP)
        c.set_batches([4, 8, 16, 36])
        nb, ch = c.rebatch([1.0, 2.0, 4.0, 9.0])
        assert nb.tolist() == [4, 8, 16, 36] and ch.tolist() == [0, 0, 0, 0]
    # uniform cluster keeps uniform batches (HL1: variable batching equals uniform batching)
    c = O.Controller(8, 256, 4, 96, 0.0, 1.0, O.MODE_BSP)
    nb, _ = c.rebatch([3.7] * 8)
    assert nb.tolist() == [32] * 8


def test_inside_deadband_no_adjustment():
    """Eq. 7: a relative change below the threshold leaves the batch alone."""
    c = O.Controller(2, 64, 4, 96, 0.10, 1.0, O.MODE_ASP)
    nb, ch = c.rebatch([1.0, 1.1])     # b* = (30.5, 33.6): changes 4.9% and 4.7%
    assert nb.tolist() == [32, 32] and ch.tolist() == [0, 0]
    c = O.Controller(2, 64, 4, 96, 0.04, 1.0, O.MODE_ASP)
    nb, ch = c.rebatch([1.0, 1.1])     # now outside the band: 30.545 -> 31, 33.6 -> 34
    assert nb.tolist() == [31, 34]


def test_deadband_threshold_is_inclusive_and_relative_to_new_value():
    """|b* - b| / b* >= deadband with b* in the denominator: b = 30, b* = 40 gives exactly 0.25."""
    # two workers, b = (30, 50), choose T so that b* = (40, 40): T tbar = 40 with t = (1, 1) -> no.
    # b* = T_k * tbar; T = (4, 4), t = (7.5, 12.5), tbar = 10 -> b* = (40, 40).
    c = O.Controller(2, 80, 1, 1000, 0.25, 1.0, O.MODE_ASP)
    c.set_batches([30, 50])
    nb, ch = c.rebatch([4.0, 4.0])
    # worker 0: |40-30|/40 = 0.25 -> adjusts (inclusive). worker 1: |40-50|/40 = 0.25 -> adjusts.
    assert nb.tolist() == [40, 40]
    c = O.Controller(2, 80, 1, 1000, 0.26, 1.0, O.MODE_ASP)
    c.set_batches([30, 50])
    nb, ch = c.rebatch([4.0, 4.0])
    assert nb.tolist() == [30, 50]
    # were the denominator the OLD batch, worker 0 (10/30 = 0.33) would have moved at 0.26
    

def test_bounds_clamp():
    c = O.Controller(2, 64, 12, 40, 0.0, 1.0, O.MODE_ASP)
    nb, _ = c.rebatch([1.0, 31.0])     # b* = (16.5.., 512) -> (17, 40)
    assert nb.tolist() == [17, 40]
    nb, _ = c.rebatch([0.01, 31.0])    # worker 0 collapses below b_min
    assert nb[0] == 12


def test_time_input_equals_throughput_input():
    T = np.array([1.5, 2.5, 4.0, 7.0])
    a = O.Controller(4, 128, 4, 96, 0.1, 1.0, O.MODE_BSP)
    b = O.Controller(4, 128, 4, 96, 0.1, 1.0, O.MODE_BSP, O.FLAG_INPUT_IS_TIME)
    for _ in range(4):
        nb_a, _ = a.rebatch(T)
        nb_b, _ = b.rebatch(b.batches / T)
        assert nb_a.tolist() == nb_b.tolist()


def test_ewma_smoothing():
    """alpha = 1 ignores history; alpha = 0.5 averages the new compute time with the old one."""
    c = O.Controller(2, 64, 1, 1000, 0.0, 0.5, O.MODE_ASP, O.FLAG_INPUT_IS_TIME)
    c.rebatch([4.0, 4.0])                       # first sample initialises: s = (4, 4); no change
    assert c.batches.tolist() == [32, 32]
    _, _, bstar = c.rebatch([8.0, 4.0], want_bstar=True)   # s = (6, 4), tbar = 5
    np.testing.assert_allclose(bstar, [32 * 5 / 6, 32 * 5 / 4], rtol=1e-14)


def test_permutation_of_workers_permutes_batches():
    rng = np.random.default_rng(5)
    for _ in range(50):
        K = 6
        T = rng.permutation(np.array([1.0, 1.7, 2.9, 4.1, 5.3, 8.0]))
        perm = rng.permutation(K)
        a = O.Controller(K, 192, 4, 96, 0.1, 1.0, O.MODE_ASP)
        b = O.Controller(K, 192, 4, 96, 0.1, 1.0, O.MODE_ASP)
        na, _ = a.rebatch(T)
        nb, _ = b.rebatch(T[perm])
        assert na[perm].tolist() == nb.tolist()


def test_static_hl8_settles_within_a_few_adjustments():
    """Sec. IV-D: from b = 32 with bounds (12, 96), dead-band 15% and no global-batch rule the
    batches reach a steady state in 2-4 adjustments under static heterogeneity."""
    c = O.Controller(4, 128, 12, 96, 0.15, 1.0, O.MODE_ASP)
    T = [6.0, 6.0, 4.0, 32.0]                    # Table I, BSP HL8 core counts
    changes = []
    for _ in range(8):
        _, ch = c.rebatch(T)
        changes.append(int(ch.any()))
    first_quiet = changes.index(0)
    assert 1 <= first_quiet <= 4 and sum(changes[first_quiet:]) == 0


def test_asp_report_waits_for_all_workers_then_recomputes_all():
    g = [c for c in GOLD["cases"] if c["mode"] == "asp"][0]
    c = O.Controller(g["K"], g["B"], g["b_min"], g["b_max"], g["deadband"], 1.0, O.MODE_ASP)
    T = g["throughput"]
    for k in range(3):
        assert c.asp_report(k, 32, T[k]) == 32          # fewer than K entries: keep the batch
    assert c.asp_report(3, 32, T[3]) == g["expect"][0][3]
    assert c.batches.tolist() == g["expect"][0]         # every entry was re-evaluated
    # no global-batch rule in ASP: the sum moved away from B
    assert c.batches.sum() != g["B"]


@pytest.mark.parametrize("case", GOLD["report_cases"], ids=lambda c: c["name"].split()[0])
def test_hand_derived_report_sequences(case):
    """Algorithm 2 evalBsz by hand: the server stores the batch the worker RAN (which need not be
    the entry it holds) and the smoothed compute time, then re-evaluates every entry."""
    flags = O.FLAG_INPUT_IS_TIME if case["input"] == "time" else 0
    c = O.Controller(case["K"], case["B"], case["b_min"], case["b_max"], case["deadband"], case["alpha"],
                     O.MODE_ASP, flags)
    assert c.batches.tolist() == case["b0"]
    for r in case["reports"]:
        assert c.asp_report(r["worker"], r["b_used"], r["measured"]) == r["returns"]
        assert c.batches.tolist() == r["map_after"]


@pytest.mark.parametrize("case", GOLD["multiplicative_cases"], ids=lambda c: c["name"].split()[0])
def test_hand_derived_traces_multiplicative_conservation(case):
    c = O.Controller(case["K"], case["B"], case["b_min"], case["b_max"], case["deadband"], 1.0, O.MODE_BSP,
                     O.FLAG_CONSERVE_MULTIPLICATIVE)
    assert c.batches.tolist() == case["b0"]
    for want in case["expect"]:
        assert c.rebatch(case["throughput"])[0].tolist() == want


def test_multiplicative_conservation_lands_on_the_proportional_split_in_one_step():
    """From equal batches, without dead-band and with wide bounds, the renormalised real-valued
    batches are B * T_k / sum(T): Eq. 4a with the throughputs as capacities."""
    rng = np.random.default_rng(11)
    for _ in range(200):
        K = int(rng.integers(2, 33))
        T = rng.uniform(0.5, 20.0, K)
        Bg = 32 * K
        c = O.Controller(K, Bg, 1, 10**6, 0.0, 1.0, O.MODE_BSP, O.FLAG_CONSERVE_MULTIPLICATIVE)
        nb, _, scaled = c.rebatch(T, want_scaled=True)
        np.testing.assert_allclose(scaled, Bg * T / T.sum(), rtol=1e-12)
        assert nb.sum() == Bg
        # and the integers are the static split's, whenever no share sits within rounding noise of a half
        frac = (Bg * T / T.sum()) % 1.0
        if np.all(np.abs(frac - 0.5) > 1e-9):
            s = O.Controller(K, Bg, 1, 10**6, 0.0, 1.0, O.MODE_BSP)
            assert nb.tolist() == s.rebatch_static(T).tolist()


def test_multiplicative_conservation_keeps_sum_and_bounds_exhaustively():
    """Every initial split of small global batches over 2-3 workers, a grid of throughputs: after
    the re-batch the sum is B and every batch is within the bounds; the asynchronous mode ignores
    the flag (no global-batch rule there)."""
    grid = [0.5, 1.0, 2.0, 3.5, 8.0]
    for K in (2, 3):
        for Bg in range(K * 2, 13):
            b_min, b_max = 2, Bg - 2 * (K - 1)
            for b0 in itertools.product(range(b_min, b_max + 1), repeat=K):
                if sum(b0) != Bg:
                    continue
                for T in itertools.product(grid, repeat=K):
                    for db in (0.0, 0.1):
                        c = O.Controller(K, Bg, b_min, b_max, db, 1.0, O.MODE_BSP, O.FLAG_CONSERVE_MULTIPLICATIVE)
                        c.set_batches(b0)
                        nb, _ = c.rebatch(T)
                        assert nb.sum() == Bg and nb.min() >= b_min and nb.max() <= b_max, (b0, T, db)
    a = O.Controller(4, 128, 4, 96, 0.1, 1.0, O.MODE_ASP, O.FLAG_CONSERVE_MULTIPLICATIVE)
    b = O.Controller(4, 128, 4, 96, 0.1, 1.0, O.MODE_ASP)
    assert a.rebatch([4, 4, 4, 28])[0].tolist() == b.rebatch([4, 4, 4, 28])[0].tolist() == [25, 25, 25, 96]


def test_equal_times_are_a_fixed_point_under_both_conservation_readings():
    for flags in (0, O.FLAG_CONSERVE_MULTIPLICATIVE):
        c = O.Controller(4, 64, 2, 48, 0.0, 1.0, O.MODE_BSP, flags)
        c.set_batches([4, 8, 16, 36])
        assert c.rebatch([1, 2, 4, 9])[0].tolist() == [4, 8, 16, 36]


def test_batches_depend_only_on_throughput_ratios():
    """Eq. 6 in the form b* = T_k * mean_j(b_j / T_j): multiplying every throughput by the same
    factor changes no batch.  With a power of two as the factor every intermediate scales exactly,
    so the integers must be identical, synchronous and asynchronous, smoothed or not."""
    rng = np.random.default_rng(21)
    for _ in range(100):
        K = int(rng.integers(2, 33))
        mode = int(rng.integers(0, 2))
        alpha = float(rng.choice([1.0, 0.5]))
        a = O.Controller(K, 32 * K, 4, 96, 0.1, alpha, mode)
        b = O.Controller(K, 32 * K, 4, 96, 0.1, alpha, mode)
        base = 8.0 ** rng.uniform(0, 1, K)
        for step in range(5):
            T = base * (1 + 0.2 * (2 * rng.uniform(0, 1, K) - 1))
            na, _ = a.rebatch(T)
            nb, _ = b.rebatch(T * 64.0)
            assert na.tolist() == nb.tolist()


def test_errors_leave_state_untouched():
    c = O.Controller(4, 64, 2, 48, 0.1)
    before = c.batches.copy()
    for bad in ([1.0, 2.0, 0.0, 1.0], [1.0, -2.0, 1.0, 1.0], [1.0, np.nan, 1.0, 1.0], [np.inf, 1, 1, 1]):
        with pytest.raises(O.OracleError) as e:
            c.rebatch(bad)
        assert e.value.code == O.ERR_MEASUREMENT
        assert c.batches.tolist() == before.tolist()
    with pytest.raises(O.OracleError):
        O.Controller(4, 64, 17, 48, 0.1)          # K * b_min > B
    with pytest.raises(O.OracleError):
        O.Controller(4, 64, 2, 15, 0.1)           # K * b_max < B
    with pytest.raises(O.OracleError):
        c.set_batches([16, 16, 16, 15])           # sum != B in BSP


def test_initial_batches_when_k_does_not_divide_b():
    c = O.Controller(3, 64, 1, 64, 0.1)
    assert c.batches.tolist() == [22, 21, 21]


def test_static_variable_batching_by_capacity():
    """Eq. 4a with the core counts of Table I: shares of B proportional to cores."""
    c = O.Controller(4, 128, 4, 96, 0.1)
    assert c.rebatch_static([12, 12, 12, 12]).tolist() == [32, 32, 32, 32]      # HL1
    assert c.rebatch_static([6, 6, 4, 32]).tolist() == [16, 16, 11, 85]         # BSP HL8: 16, 16, 10.67, 85.33
    assert c.rebatch_static([10, 10, 6, 22]).tolist() == [27, 27, 16, 58]       # 26.67->27, 16, 58.67->59: 1 over, from the largest
    c3 = O.Controller(3, 64, 1, 64, 0.1)
    assert c3.rebatch_static([1, 1, 1]).tolist() == [22, 21, 21]                # 21.33 each, one unit short -> lowest index
    rng = np.random.default_rng(7)
    for _ in range(100):
        K = int(rng.integers(2, 17))
        cc = O.Controller(K, 32 * K, 4, 96, 0.1)
        nb = cc.rebatch_static(rng.uniform(1, 8, K))
        assert nb.sum() == 32 * K and nb.min() >= 4 and nb.max() <= 96
