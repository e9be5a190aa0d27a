"""Pins for the oracle's sampler algebra and speculation bookkeeping (CPU only).

Every check compares an oracle function against something fixed outside it:
a closed form, an identity between two of the paper's own equations, or a
brute-force definition written here."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import nfd_oracle as O
from paper_2506_01380_b200 import inputs as I

RNG = np.random.default_rng(123)
TPS = [0.0, 0.05, math.pi / 8, math.pi / 4, 1.0, 3 * math.pi / 8, 1.5, math.pi / 2]


def test_fm_time_closed_forms():
    # Section 4.1: t = sin t'/(sin t' + cos t'); values at 0, pi/4, pi/2 are 0, 1/2, 1.
    assert O.fm_time(0.0) == 0.0
    assert abs(O.fm_time(math.pi / 4) - 0.5) < 1e-15
    assert abs(O.fm_time(math.pi / 2) - 1.0) < 1e-15
    for tp in TPS[:-1]:
        # equivalent form tan/(1+tan)
        assert abs(O.fm_time(tp) - math.tan(tp) / (1 + math.tan(tp))) < 1e-14


@pytest.mark.parametrize("tp", TPS)
def test_fm_input_is_the_flow_matching_interpolant(tp):
    # TrigFlow sample x' = cos t' x0 + sin t' sigma_d z.  Rescaled by the paper's
    # factor it must be Flow Matching's interpolant (1-t) x0/sigma_d + t z (Eq. 1).
    sd = 0.37
    x0, z = RNG.standard_normal(50), RNG.standard_normal(50)
    xp = math.cos(tp) * x0 + math.sin(tp) * sd * z
    t = O.fm_time(tp)
    want = (1 - t) * x0 / sd + t * z
    np.testing.assert_allclose(O.fm_input(xp, tp, sd), want, atol=1e-13)
    # sqrt(t^2+(1-t)^2) = 1/(sin+cos)
    assert abs(math.sqrt(t * t + (1 - t) ** 2) - 1 / (math.sin(tp) + math.cos(tp))) < 1e-14


@pytest.mark.parametrize("tp", TPS)
def test_F_theta_is_trigflow_velocity(tp):
    # With eps_hat = x^t + (1-t) v and x0_hat = x^t - t v (Section 3.2), the
    # TrigFlow target is cos t' * eps_hat - sin t' * x0_hat.
    t = O.fm_time(tp)
    x, v = RNG.standard_normal(40), RNG.standard_normal(40)
    want = math.cos(tp) * (x + (1 - t) * v) - math.sin(tp) * (x - t * v)
    np.testing.assert_allclose(O.F_theta(x, v, t), want, atol=1e-13)


@pytest.mark.parametrize("tp", TPS)
def test_f_theta_collapses_and_recovers_x0(tp):
    sd = 0.5
    t = O.fm_time(tp)
    x0, z = RNG.standard_normal(64), RNG.standard_normal(64)
    xp = O.renoise(x0, z, tp, sd)
    x_in = O.fm_input(xp, tp, sd)
    v_true = z - x0 / sd                      # Eq. 1's target velocity, in sigma_d units
    got = O.f_theta(xp, O.F_theta(x_in, v_true, t), tp, sd)
    np.testing.assert_allclose(got, x0, atol=1e-12)          # exact velocity => exact clean frame
    # and for an arbitrary velocity it equals sigma_d (x^t - t v)
    v = RNG.standard_normal(64)
    got = O.f_theta(xp, O.F_theta(x_in, v, t), tp, sd)
    np.testing.assert_allclose(got, sd * (x_in - t * v), atol=1e-12)


@pytest.mark.parametrize("tp", TPS[:-1])
def test_section32_formula_agrees(tp):
    t = O.fm_time(tp)
    x, v = RNG.standard_normal(30), RNG.standard_normal(30)
    np.testing.assert_allclose(O.x0_from_velocity(x, v, t), x - t * v, atol=1e-11)


def test_schedule():
    # 4 steps, linear between pi/2 and 0, evaluated at pi/2, 3pi/8, pi/4, pi/8.
    s = O.trig_schedule(4)
    np.testing.assert_allclose(s, [math.pi / 2, 3 * math.pi / 8, math.pi / 4, math.pi / 8], atol=1e-15)
    assert O.fm_time(s[0]) == pytest.approx(1.0, abs=1e-15)


def test_accepted_count_brute_force():
    for n in range(1, 7):
        for acts in itertools.product([0, 1], repeat=n):
            for k in range(1, 5):
                for i in range(n):
                    # definition: smallest j>=1 with a different action, capped at k and at the end
                    want = None
                    for j in range(1, k):
                        if i + j >= n or acts[i + j] != acts[i]:
                            want = j
                            break
                    if want is None:
                        want = k
                    assert O.accepted_count(list(acts), i, k) == want


def test_expected_acceptance_closed_form():
    # Markov chain with repeat probability p: E[accepted per pass of k] = (1-p^k)/(1-p).
    cfg = I.make_cfg("nfd310m")
    p, k = 0.8, 4
    acts = I.make_action_chain(cfg, 60000, seed=0, p_repeat=p)
    i = tot = passes = 0
    while i + k < len(acts):
        n = O.accepted_count(acts, i, k)
        tot += n
        passes += 1
        i += n
    want = (1 - p ** k) / (1 - p)
    assert abs(want - 2.952) < 1e-3
    assert abs(tot / passes - want) < 0.03
    # empirical repeat probability of the generator
    rep = np.mean(acts[1:] == acts[:-1])
    assert abs(rep - p) < 0.01


def test_paper_shape_facts():
    # tests/golden/paper_shapes.txt: numbers the paper prints (tokens per frame,
    # the appendix size table).
    here = os.path.dirname(__file__)
    rows = {}
    for line in open(os.path.join(here, "golden", "paper_shapes.txt")):
        line = line.split("#")[0].strip()
        if line:
            k, *v = line.split()
            rows[k] = [int(x) for x in v]
    cfg = I.make_cfg("nfd310m")
    th, tw = rows["tokens_grid"]
    assert (cfg["latent_h"] // cfg["patch"], cfg["latent_w"] // cfg["patch"]) == (th, tw)
    assert I.tokens_per_frame(cfg) == rows["tokens_per_frame"][0] == th * tw
    for name in ("paper130m", "paper310m", "paper774m"):
        c = I.make_cfg(name)
        assert [c["d_model"], c["d_mlp"], c["n_heads"], c["n_layers"]] == rows[name]


# ---------------------------------------------------------------- DPM-Solver++(2M) on the Flow-Matching path
def test_dpmpp_is_exact_for_a_constant_data_prediction():
    """A data-prediction solver integrates exactly when x0_theta does not change along the path: the result
    is that constant whatever the number of evaluations and whatever the start."""
    rng = np.random.default_rng(0)
    c, xT = rng.standard_normal(7), rng.standard_normal(7)
    for n in (1, 2, 3, 5, 18):
        np.testing.assert_allclose(O.dpmpp_2m(lambda x, t: c, xT, n), c, atol=1e-13)


def test_dpmpp_coefficients_match_the_published_form():
    """a = sigma_t/sigma_s, b = -alpha_t (e^{-h} - 1), 1/(2r) = h/(2 h_prev) with lambda = ln(alpha/sigma), on
    interior steps; the limits at both ends: first step from t = 1 is x_t = t x_1 + (1-t) x0 (first order),
    the second step has no finite previous step (c = 0), the last step to t = 0 returns the data prediction."""
    lam = lambda u: math.log((1 - u) / u)
    for (t2, t1, t0) in ((0.9, 0.8, 0.7), (0.5, 0.45, 0.2), (0.3, 0.2, 0.1)):
        a, b, c = O.dpmpp_coeffs(t2, t1, t0, last=False)
        h, hp = lam(t0) - lam(t1), lam(t1) - lam(t2)
        assert abs(a - t0 / t1) < 1e-15
        assert abs(b - (-(1 - t0) * (math.exp(-h) - 1))) < 1e-13
        assert abs(c - h / (2 * hp)) < 1e-15 and abs(c - 1 / (2 * (hp / h))) < 1e-13
    a, b, c = O.dpmpp_coeffs(None, 1.0, 0.75, last=False)
    assert (a, b, c) == (0.75, 0.25, 0.0)
    assert O.dpmpp_coeffs(1.0, 0.75, 0.5, last=False)[2] == 0.0
    assert O.dpmpp_coeffs(0.2, 0.1, 0.0, last=True) == (0.0, 1.0, 0.0)
    g = O.dpmpp_grid(18)
    assert len(g) == 19 and g[0] == 1.0 and g[-1] == 0.0 and abs(g[1] - 17 / 18) < 1e-15


def test_dpmpp_converges_on_gaussian_data_and_beats_the_first_order_solver():
    """Data N(mu, s^2) per element: the optimal data prediction is linear in x,
    x0*(x, t) = mu + alpha s^2 (x - alpha mu) / (alpha^2 s^2 + sigma^2), and the probability-flow ODE carries
    the start eps at t = 1 to mu + s eps at t = 0.  The solver must approach that value as the grid is refined,
    faster than first order (halving the step cuts the error by more than two; the grid's end points, where
    lambda is infinite, keep it below the factor four of a uniform-lambda grid), and it must beat the
    first-order solver (the same update with c = 0, written out here) on the same grid."""
    rng = np.random.default_rng(1)
    mu, sd = rng.standard_normal(9), 0.3 + rng.random(9)
    eps = rng.standard_normal(9)

    def x0_fn(x, t):
        al, sg = 1 - t, t
        return mu + al * sd ** 2 * (x - al * mu) / (al ** 2 * sd ** 2 + sg ** 2)

    def first_order(n):
        x = eps.copy()
        for i in range(n):
            s_, t_ = 1 - i / n, 1 - (i + 1) / n
            x = (t_ / s_) * x + ((1 - t_) - (1 - s_) * t_ / s_) * x0_fn(x, s_)
        return x

    want = mu + sd * eps
    errs = [np.abs(O.dpmpp_2m(x0_fn, eps, n) - want).max() for n in (18, 36, 72, 144)]
    assert errs[0] < 2e-2 and errs[3] < errs[2] < errs[1] < errs[0]
    for a, b in zip(errs, errs[1:]):
        assert 2.2 < a / b < 5.0, errs
    e1 = np.abs(first_order(18) - want).max()
    assert errs[0] < 0.5 * e1, (errs[0], e1)
