"""Pins for the checker's optimizer: closed forms and the paper's
state-transition recurrences.  CPU only."""
import os

import numpy as np
import pytest
import torch

from oracle import StageOptimizer, sc_coefficients

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_sc_coefficient_table():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "sc_coefficients.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 6
    for m, D, a, b in rows:
        got_a, got_b = sc_coefficients(float(m), int(D))
        assert got_a == pytest.approx(float(a), rel=1e-12, abs=1e-15)
        assert got_b == pytest.approx(float(b), rel=1e-12, abs=1e-15)


@pytest.mark.parametrize("m", [0.0, 0.5, 0.9, 0.99])
@pytest.mark.parametrize("D", [0, 1, 6, 30, 106])
def test_total_contribution_is_unchanged(m, D):
    # Section "Spike Compensation": the total contribution of a gradient over
    # training is the same as without delay: a/(1-m) + b = 1/(1-m).
    a, b = sc_coefficients(m, D)
    assert a / (1 - m) + b == pytest.approx(1 / (1 - m), rel=1e-12)


def test_zero_delay_is_sgdm_torch():
    # For D = 0 SC_D reduces to SGDM, and T = 0 predicts the weights themselves.
    rng = np.random.default_rng(0)
    w0 = rng.standard_normal(17)
    opt = StageOptimizer(w0, lr=0.03, m=0.9, delay=0, use_sc=True, use_lwp=True)
    p = torch.nn.Parameter(torch.tensor(w0, dtype=torch.float64))
    ref = torch.optim.SGD([p], lr=0.03, momentum=0.9)
    for _ in range(25):
        g = rng.standard_normal(17)
        np.testing.assert_array_equal(opt.predicted(), opt.w)
        opt.update(g)
        p.grad = torch.tensor(g, dtype=torch.float64)
        ref.step()
        np.testing.assert_allclose(opt.w, p.detach().numpy(), rtol=1e-13, atol=1e-15)


@pytest.mark.parametrize("D", [0, 1, 4, 9])
def test_impulse_response(D):
    # One gradient g arrives, zeros afterwards.  With SC_D the first step moves
    # the weight by eta * sum_{k=0..D} m^k g (the missed D terms plus its own),
    # later step k by eta * m^(D+k) g, and everything sums to eta g / (1 - m).
    lr, m, g = 0.1, 0.8, 2.5
    opt = StageOptimizer(np.zeros(1), lr, m, D, use_sc=True, use_lwp=False)
    steps, prev = [], 0.0
    for k in range(400):
        opt.update(np.array([g if k == 0 else 0.0]))
        steps.append(prev - opt.w[0])
        prev = opt.w[0]
    assert steps[0] == pytest.approx(lr * g * sum(m ** k for k in range(D + 1)), rel=1e-12)
    for k in range(1, 20):
        assert steps[k] == pytest.approx(lr * g * m ** (D + k), rel=1e-11)
    assert sum(steps) == pytest.approx(lr * g / (1 - m), rel=1e-10)
    # without compensation the same gradient's step k is eta m^k g
    plain = StageOptimizer(np.zeros(1), lr, m, D, use_sc=False, use_lwp=False)
    plain.update(np.array([g]))
    assert -plain.w[0] == pytest.approx(lr * g, rel=1e-14)


def test_velocity_and_weight_forms_agree_without_sc():
    # For unmodified SGDM, w - eta T v == w + T (w - w_prev).
    rng = np.random.default_rng(1)
    w0 = rng.standard_normal(9)
    ov = StageOptimizer(w0, 0.05, 0.9, 6, use_sc=False, use_lwp=True)
    ow = StageOptimizer(w0, 0.05, 0.9, 6, use_sc=False, use_lwp=True, w_form=True)
    for _ in range(12):
        g = rng.standard_normal(9)
        ov.update(g)
        ow.update(g)
        np.testing.assert_allclose(ov.predicted(), ow.predicted(), rtol=1e-12, atol=1e-14)
    # and with SC on they differ (Section "Combined Mitigation")
    sv = StageOptimizer(w0, 0.05, 0.9, 6)
    sw = StageOptimizer(w0, 0.05, 0.9, 6, w_form=True)
    g = rng.standard_normal(9)
    sv.update(g)
    sw.update(g)
    assert np.abs(sv.predicted() - sw.predicted()).max() > 1e-3


def test_horizon_zero_predicts_current_weights():
    opt = StageOptimizer(np.ones(3), 0.1, 0.9, 5, use_sc=False, use_lwp=False)
    opt.update(np.array([1.0, -2.0, 0.5]))
    np.testing.assert_array_equal(opt.predicted(), opt.w)


def _run_delayed(lam, lr, m, D, a, b, T, w_form, steps, w0=1.0):
    """Scalar optimizer fed g_t = lam * w_hat made at time t - D."""
    opt = StageOptimizer(np.array([w0]), lr, m, D, use_sc=False, use_lwp=True,
                         w_form=w_form, horizon=T)
    opt.a, opt.b = a, b
    preds, traj = [], [w0]
    for t in range(steps):
        preds.append(opt.predicted()[0])
        w_hat = preds[t - D] if t - D >= 0 else w0
        opt.update(np.array([lam * w_hat]))
        traj.append(opt.w[0])
    return np.array(traj)


def _recurrence(lam, lr, m, D, a, b, T, steps, w0=1.0):
    """Direct iteration of the state-transition equation (Appendix "State
    Transition Equations"): w_{t+1} = (1+m) w_t - m w_{t-1}
    - eta (a+b) g_t + eta m b g_{t-1}, g_t = lam ((T+1) w_{t-D} - T w_{t-D-1}),
    with w_k = w0 for k <= 0 and no gradient before time 0."""
    w = {k: w0 for k in range(-D - 3, 1)}

    def g(t):
        if t < 0:
            return 0.0
        return lam * ((T + 1) * w[t - D] - T * w[t - D - 1])
    for t in range(steps):
        w[t + 1] = (1 + m) * w[t] - m * w[t - 1] - lr * (a + b) * g(t) + lr * m * b * g(t - 1)
    return np.array([w[t] for t in range(steps + 1)])


@pytest.mark.parametrize("D", [0, 1, 3, 7])
def test_state_transition_sgdm_gsc_lwp(D):
    lam, lr, m, n = 0.7, 0.05, 0.9, 60
    a, b = sc_coefficients(m, D)
    # SGDM with delay: a=1, b=0, T=0
    np.testing.assert_allclose(_run_delayed(lam, lr, m, D, 1, 0, 0, False, n),
                               _recurrence(lam, lr, m, D, 1, 0, 0, n), rtol=1e-10, atol=1e-13)
    # GSC: T=0
    np.testing.assert_allclose(_run_delayed(lam, lr, m, D, a, b, 0, False, n),
                               _recurrence(lam, lr, m, D, a, b, 0, n), rtol=1e-10, atol=1e-13)
    # LWP (velocity form, no SC): a=1, b=0, T=D
    np.testing.assert_allclose(_run_delayed(lam, lr, m, D, 1, 0, D, False, n),
                               _recurrence(lam, lr, m, D, 1, 0, D, n), rtol=1e-10, atol=1e-13)
    # LWP^w + GSC
    np.testing.assert_allclose(_run_delayed(lam, lr, m, D, a, b, D, True, n),
                               _recurrence(lam, lr, m, D, a, b, D, n), rtol=1e-10, atol=1e-13)


def test_velocity_form_with_sc_differs_from_w_form_recurrence():
    # The paper analyses only the w-form of the combination because the v-form
    # has no such simple recurrence; a v-form run must not satisfy it.
    lam, lr, m, D, n = 0.7, 0.05, 0.9, 3, 40
    a, b = sc_coefficients(m, D)
    v = _run_delayed(lam, lr, m, D, a, b, D, False, n)
    r = _recurrence(lam, lr, m, D, a, b, D, n)
    assert np.abs(v - r).max() > 1e-4
