"""Pins of the oracle's aggregation and update rules (Eq. 4b/4c, Eq. 5b) against hand-computed
dyadic cases, a library optimiser, plain means, and the double-precision definition."""
import json
from pathlib import Path

import numpy as np
import pytest
import torch

from oracle import oracle as O

GOLD = json.loads((Path(__file__).parent / "golden" / "update_cases.json").read_text())


def _f(a, dt):
    return np.array(a, dtype=dt)


@pytest.mark.parametrize("name", ["bsp", "bsp_weight_decay"])
@pytest.mark.parametrize("prec", ["f32", "f64"])
def test_hand_computed_bsp_steps(name, prec):
    c = GOLD[name]
    dt = np.float32 if prec == "f32" else np.float64
    step = O.bsp_step_f32 if prec == "f32" else O.bsp_step_f64
    g = [_f(x, np.float32) for x in c["g"]]
    theta = _f(c["theta0"], dt)
    v = np.zeros(2, dt)
    for want in c["steps"]:
        sq = step(g, c["b"], theta, v, c["lr"], c["momentum"], c["weight_decay"])
        assert v.tolist() == want["v"] and theta.tolist() == want["theta"]
        if "sqnorm" in c:
            assert sq == c["sqnorm"]
    if "lambda" in c:
        l64, l32 = O.bsp_weights(c["b"])
        assert l64.tolist() == c["lambda"] and l32.tolist() == c["lambda"]


def test_hand_computed_asp_arrival():
    c = GOLD["asp"]
    assert O.asp_lr(c["lr"], c["b_used"], c["B"]) == c["eta_k"]
    for dt, fn in ((np.float32, O.asp_apply_f32), (np.float64, O.asp_apply_f64)):
        theta = _f(c["theta0"], dt)
        fn(_f(c["g"], np.float32), c["b_used"], c["B"], theta, None, c["lr"], 0.0, 0.0)
        assert theta.tolist() == c["theta"]


def _rand_case(rng, K, n, bf16=False):
    g = [rng.normal(0, 1e-3, n).astype(np.float32) for _ in range(K)]
    if bf16:
        g = [torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy() for x in g]
    theta = rng.normal(0, 0.05, n)
    b = rng.integers(1, 97, K).astype(np.int32)
    return g, theta, b


def _as_f64(g):
    if g[0].dtype == np.uint16:
        return np.stack([torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).double().numpy() for x in g])
    return np.stack([x.astype(np.float64) for x in g])


@pytest.mark.parametrize("K", [1, 3, 16])
@pytest.mark.parametrize("bf16", [False, True])
def test_f64_matches_library_optimizer(K, bf16):
    """gbar from a library contraction, the update from torch.optim.SGD (momentum, weight decay,
    dampening 0, no Nesterov) in double, over several steps.  K = 1 is vanilla SGD-momentum."""
    rng = np.random.default_rng(10 + K)
    n = 1000
    g, theta0, b = _rand_case(rng, K, n, bf16)
    lam = torch.tensor(b, dtype=torch.float64) / float(b.sum())
    G = torch.from_numpy(_as_f64(g))
    p = torch.nn.Parameter(torch.from_numpy(theta0.copy()))
    opt = torch.optim.SGD([p], lr=0.1, momentum=0.9, weight_decay=5e-4)
    theta = theta0.copy()
    v = np.zeros(n)
    for _ in range(5):
        p.grad = torch.tensordot(lam, G, dims=1)
        opt.step()
        sq = O.bsp_step_f64(g, b, theta, v, 0.1, 0.9, 5e-4)
        np.testing.assert_allclose(theta, p.detach().numpy(), rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(sq, float((p.grad ** 2).sum()), rtol=1e-12)
    if K == 1:
        assert O.bsp_weights(b)[0].tolist() == [1.0]


def test_plain_sgd_when_no_momentum_no_decay():
    """mu = wd = 0 is Eq. 4c itself: theta - eta * sum_k lambda_k g_k; the momentum buffer may be absent."""
    rng = np.random.default_rng(20)
    g, theta0, b = _rand_case(rng, 5, 777)
    theta = theta0.copy()
    O.bsp_step_f64(g, b, theta, None, 0.3, 0.0, 0.0)
    want = theta0 - 0.3 * (b[:, None] / b.sum() * _as_f64(g)).sum(0)
    np.testing.assert_allclose(theta, want, rtol=1e-13, atol=1e-16)


@pytest.mark.parametrize("K", [2, 4, 8, 16, 32])
def test_equal_batches_reduce_to_plain_mean(K):
    rng = np.random.default_rng(30 + K)
    g, theta0, _ = _rand_case(rng, K, 513)
    b = np.full(K, 7, np.int32)
    l64, l32 = O.bsp_weights(b)
    assert (l64 == 1.0 / K).all() and (l32 == np.float32(1.0 / K)).all()
    theta = theta0.copy()
    O.bsp_step_f64(g, b, theta, None, 1.0, 0.0, 0.0)
    np.testing.assert_allclose(theta0 - theta, _as_f64(g).mean(0), rtol=1e-12, atol=1e-16)


def test_unscaled_mean_flag_ignores_batches():
    rng = np.random.default_rng(40)
    g, theta0, b = _rand_case(rng, 6, 300)
    theta = theta0.copy()
    O.bsp_step_f64(g, b, theta, None, 1.0, 0.0, 0.0, flags=O.FLAG_UNSCALED_MEAN)
    np.testing.assert_allclose(theta0 - theta, _as_f64(g).mean(0), rtol=1e-12, atol=1e-16)
    # and the weighted result differs from it when the batches are unequal
    theta2 = theta0.copy()
    O.bsp_step_f64(g, b, theta2, None, 1.0, 0.0, 0.0)
    assert np.abs(theta2 - theta).max() > 1e-6


def test_weights_sum_to_one_and_are_proportional():
    rng = np.random.default_rng(41)
    for _ in range(100):
        K = int(rng.integers(1, 33))
        b = rng.integers(1, 97, K).astype(np.int32)
        l64, l32 = O.bsp_weights(b)
        assert abs(l64.sum() - 1.0) < 1e-14
        np.testing.assert_allclose(l64 * b.sum(), b, rtol=1e-15)
        assert (l32 == l64.astype(np.float32)).all()


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("K", [1, 4, 16, 32])
def test_f32_mode_stays_within_rounding_of_the_definition(K, bf16):
    """Single-precision mode vs the double definition after 10 steps: the only differences are
    the float rounding of lambda and of each fused multiply-add."""
    rng = np.random.default_rng(50 + K)
    n = 4099
    g, theta0, b = _rand_case(rng, K, n, bf16)
    t32, v32 = theta0.astype(np.float32), np.zeros(n, np.float32)
    t64, v64 = t32.astype(np.float64), np.zeros(n)
    for _ in range(10):
        s32 = O.bsp_step_f32(g, b, t32, v32, 0.1, 0.9, 1e-4)
        s64 = O.bsp_step_f64(g, b, t64, v64, 0.1, 0.9, 1e-4)
        assert abs(s32 - s64) <= 1e-5 * s64
    np.testing.assert_allclose(t32, t64, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(v32, v64, rtol=1e-5, atol=1e-8)
    assert np.abs(t32 - t64).max() > 0        # it is a different arithmetic, not a copy


def test_f32_mode_is_an_ordered_fma_chain():
    """Worker order matters in float: build a case where ascending-order FMAs give a different
    bit pattern than the reverse order, and check the oracle gives the ascending result
    (computed here with exact rational arithmetic rounded once per FMA)."""
    from fractions import Fraction

    def fma_f32(a, b, c):
        exact = Fraction(float(a)) * Fraction(float(b)) + Fraction(float(c))
        # round the exact rational to float32: go through float64 only when that is exact enough;
        # numpy rounds float64 -> float32 correctly, and the exact value here fits in 53 bits.
        f = float(exact)
        assert Fraction(f) == exact
        return np.float32(f)

    lam_b = np.array([1, 2, 1], np.int32)                 # lambda = (0.25, 0.5, 0.25)
    g = [np.array([x], np.float32) for x in (2.0 ** 26, -(2.0 ** 25), 1.0)]   # terms 2^24, -2^24, 0.25
    lam = O.bsp_weights(lam_b)[1]
    acc = np.float32(0)
    for k in range(3):
        acc = fma_f32(lam[k], g[k][0], acc)
    rev = np.float32(0)
    for k in (2, 1, 0):
        rev = fma_f32(lam[k], g[k][0], rev)
    theta = np.zeros(1, np.float32)
    O.bsp_step_f32(g, lam_b, theta, None, 1.0, 0.0, 0.0)
    assert acc == np.float32(0.25) and rev == np.float32(0.0)
    assert -theta[0] == acc


def test_bf16_conversions_match_library_cast():
    allbits = np.arange(65536, dtype=np.uint16)
    want = torch.from_numpy(allbits.view(np.int16)).view(torch.bfloat16).float().numpy()
    got = O.bf16_to_float(allbits)
    assert (got.view(np.uint32) == want.view(np.uint32)).all()
    rng = np.random.default_rng(60)
    x = np.concatenate([
        rng.normal(0, 1, 100000).astype(np.float32),
        rng.integers(0, 2 ** 32, 200000, dtype=np.uint64).astype(np.uint32).view(np.float32),
        np.array([0.0, -0.0, np.inf, -np.inf, 1.00390625, 1.01171875, 3.3895314e38, 1e-40], np.float32),
    ])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = O.float_to_bf16(x)
    finite = ~np.isnan(x)
    assert (got[finite] == want[finite]).all()
    nan_out = O.bf16_to_float(got[~finite])
    assert np.isnan(nan_out).all()


def test_low_precision_copy_is_rounded_parameter():
    rng = np.random.default_rng(70)
    g, theta0, b = _rand_case(rng, 4, 1001, bf16=True)
    theta = theta0.astype(np.float32)
    v = np.zeros(1001, np.float32)
    lp = np.zeros(1001, np.uint16)
    O.bsp_step_f32(g, b, theta, v, 0.1, 0.9, 0.0, theta_lp=lp)
    want = torch.from_numpy(theta).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (lp == want).all()


def test_asp_learning_rate_scaling():
    assert O.asp_lr(0.1, 32, 512) == 0.1 * 32 / 512
    assert O.asp_lr(0.1, 128, 128) == 0.1                        # one worker holding all of B
    assert O.asp_lr(0.8, 16, 64) == 0.8 / 4                      # b = B/K -> eta/K
    assert O.asp_lr(0.1, 32, 512, O.FLAG_ASP_NO_LR_SCALE) == 0.1


@pytest.mark.parametrize("mu", [0.0, 0.9])
def test_asp_matches_library_optimizer_with_scaled_lr(mu):
    rng = np.random.default_rng(80)
    n = 500
    theta0 = rng.normal(0, 0.05, n)
    p = torch.nn.Parameter(torch.from_numpy(theta0.copy()))
    opt = torch.optim.SGD([p], lr=1.0, momentum=mu, weight_decay=1e-3)
    theta = theta0.copy()
    v = np.zeros(n) if mu else None
    for step in range(6):
        b_used = int(rng.integers(4, 97))
        g = rng.normal(0, 1e-3, n).astype(np.float32)
        for grp in opt.param_groups:
            grp["lr"] = 0.1 * b_used / 512
        p.grad = torch.from_numpy(g.astype(np.float64))
        opt.step()
        O.asp_apply_f64(g, b_used, 512, theta, v, 0.1, mu, 1e-3)
        np.testing.assert_allclose(theta, p.detach().numpy(), rtol=1e-12, atol=1e-16)


def test_asp_f32_within_rounding_of_definition():
    rng = np.random.default_rng(90)
    n = 3001
    t32 = rng.normal(0, 0.05, n).astype(np.float32)
    t64 = t32.astype(np.float64)
    for _ in range(20):
        g = rng.normal(0, 1e-3, n).astype(np.float32)
        b_used = int(rng.integers(4, 97))
        O.asp_apply_f32(g, b_used, 512, t32, None, 0.1, 0.0, 0.0)
        O.asp_apply_f64(g, b_used, 512, t64, None, 0.1, 0.0, 0.0)
    np.testing.assert_allclose(t32, t64, rtol=1e-6, atol=1e-7)


def test_staleness_is_tallied_not_applied():
    s = O.TauStats()
    for tau in (0, 0, 5, 31, 32, 100):
        s.record(tau)
    assert s.hist[0] == 2 and s.hist[5] == 1 and s.hist[31] == 1 and s.hist[32] == 2
    assert s.hist.sum() == 6 and s.tau_max == 100


def test_overwrite_semantics_hand_case():
    """Algorithm 2 literally: a push replaces the server copy by snapshot - eta_k g, so what
    arrived since the worker's pull is lost; applying the same gradients instead keeps both."""
    c = GOLD["asp_overwrite"]
    for dt, push, apply_ in ((np.float32, O.asp_push_overwrite_f32, O.asp_apply_f32),
                             (np.float64, O.asp_push_overwrite_f64, O.asp_apply_f64)):
        theta = _f(c["theta0"], dt)
        applied = _f(c["theta0"], dt)
        for ev in c["events"]:
            push(_f(ev["g"], np.float32), ev["b_used"], c["B"], theta, _f(ev["snapshot"], dt), c["lr"])
            assert theta.tolist() == ev["theta_after"]
            apply_(_f(ev["g"], np.float32), ev["b_used"], c["B"], applied, None, c["lr"], 0.0, 0.0)
        assert applied.tolist() == c["apply_semantics_would_give"]


def test_overwrite_equals_apply_when_nothing_arrived_in_between():
    rng = np.random.default_rng(91)
    n = 2001
    g = rng.normal(0, 1e-3, n).astype(np.float32)
    for dt, push, apply_ in ((np.float32, O.asp_push_overwrite_f32, O.asp_apply_f32),
                             (np.float64, O.asp_push_overwrite_f64, O.asp_apply_f64)):
        server = rng.normal(0, 0.05, n).astype(dt)
        a, b = server.copy(), server.copy()
        push(g, 24, 512, a, server.copy(), 0.1, 1e-3)
        apply_(g, 24, 512, b, None, 0.1, 0.0, 1e-3)
        assert np.array_equal(a, b)


def test_overwrite_ignores_the_current_server_copy():
    rng = np.random.default_rng(92)
    n = 500
    g = rng.normal(0, 1e-3, n).astype(np.float32)
    snap = rng.normal(0, 0.05, n)
    out1, out2 = rng.normal(0, 1, n), np.zeros(n)
    O.asp_push_overwrite_f64(g, 16, 128, out1, snap, 0.1)
    O.asp_push_overwrite_f64(g, 16, 128, out2, snap, 0.1)
    assert np.array_equal(out1, out2)
    np.testing.assert_allclose(out1, snap - 0.1 * 16 / 128 * g.astype(np.float64), rtol=1e-14, atol=1e-18)
