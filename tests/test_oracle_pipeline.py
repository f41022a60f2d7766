"""Pins for the checker's pipeline schedule.  CPU only.

None of these re-run the checker against itself: the references are a torch
SGD loop, a torch forward pass, integer schedule arithmetic from the paper's
appendix, and a per-sample replay of every gradient with torch autograd."""
import math

import numpy as np
import pytest
import torch

from oracle import PBOracle, sc_coefficients
from pb_workloads import (he_normal_weights, make_inputs, mlp, tiny_cnn, tiny_resnet,
                          workload, Layer, OP, Workload, preact_resnet)
from tests import torch_ref


def _oracle(wl, record=False, lr=None, flags=None, **kw):
    o = PBOracle(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes,
                 wl.lr if lr is None else lr, wl.momentum,
                 wl.flags if flags is None else flags, record=record, **kw)
    o.set_weights(he_normal_weights(wl.seed, wl))
    return o


def _thetas(stages, flat):
    out, off = [], 0
    for st in stages:
        out.append(torch.tensor(np.asarray(flat[off:off + st.n_params]), dtype=torch.float64))
        off += st.n_params
    return out


def test_single_stage_is_plain_sgdm():
    # S = 1: delay 2(S-1-0) = 0, so PB+SC+LWP must be batch-1 SGD with momentum.
    wl = mlp([12, 7], lr=0.05, seed=5)
    assert wl.n_stages == 1
    o = _oracle(wl)
    w0 = he_normal_weights(wl.seed, wl).astype(np.float64)
    W = torch.nn.Parameter(torch.tensor(w0[:84]).view(7, 12))
    b = torch.nn.Parameter(torch.tensor(w0[84:]))
    ref = torch.optim.SGD([W, b], lr=0.05, momentum=0.9)
    x, y = make_inputs(wl.seed, 30, 12, 7)
    for t in range(30):
        loss = o.tick(x[t], y[t])
        ref.zero_grad()
        lt = torch.nn.functional.cross_entropy(
            (W @ torch.tensor(x[t], dtype=torch.float64) + b)[None], torch.tensor([int(y[t])]))
        lt.backward()
        ref.step()
        assert loss == pytest.approx(lt.item(), rel=1e-12)
        got = o.get_weights()
        np.testing.assert_allclose(got[:84], W.detach().numpy().ravel(), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(got[84:], b.detach().numpy(), rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("make", [lambda: mlp([10, 8, 6, 4]), tiny_cnn, tiny_resnet,
                                  lambda: tiny_resnet(bottleneck=True), preact_resnet])
def test_latency_and_frozen_forward(make):
    # A sample takes 2S-1 steps; its loss appears S-1 ticks after it enters.
    # With lr = 0 the weights never move, so the loss at tick t is an ordinary
    # forward pass of the fixed network on sample t-(S-1).
    wl = make()
    o = _oracle(wl, lr=0.0)
    S = wl.n_stages
    stages = torch_ref.build(wl)
    th = _thetas(stages, he_normal_weights(wl.seed, wl))
    n = 2 * S + 3
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    for t in range(n):
        loss = o.tick(x[t], y[t])
        if t < S - 1:
            assert math.isnan(loss)
        else:
            i = t - (S - 1)
            xt = torch.tensor(x[i], dtype=torch.float64).view(*wl.in_shape)
            assert loss == pytest.approx(torch_ref.network_loss(stages, th, xt, y[i]).item(), rel=1e-10)
    np.testing.assert_array_equal(o.get_weights(), he_normal_weights(wl.seed, wl).astype(np.float64))


@pytest.mark.parametrize("make", [lambda: mlp([10, 8, 6, 5, 4]), tiny_resnet])
def test_staleness_equals_stage_delay(make):
    # Eq. (F_i): the forward weights of sample i at stage s are 2(S-1-s)
    # updates older than its backward weights, once the stage has begun updating.
    wl = make()
    o = _oracle(wl, record=True)
    S = wl.n_stages
    n = 4 * S
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    for t in range(n):
        o.tick(x[t], y[t])
    checked = 0
    for (s, i), bv in o.bwd_version.items():
        fv = o.fwd_version[(s, i)]
        first_update_tick = 2 * (S - 1) - s
        assert bv == i                       # sample i's gradient is update number i
        if i + s >= first_update_tick:
            assert bv - fv == 2 * (S - 1 - s) == o.delay(s)
            checked += 1
        else:
            assert fv == 0
    assert checked > S
    # a sample needs 2S-1 ticks: sample i is back at stage 0 at tick i+2(S-1)
    assert max(i for (s, i) in o.bwd_version if s == 0) == n - 1 - 2 * (S - 1)


@pytest.mark.parametrize("make,flags", [
    (lambda: mlp([9, 7, 6, 5], lr=0.05), 3), (tiny_cnn, 3), (tiny_resnet, 3),
    (lambda: tiny_resnet(bottleneck=True), 3), (tiny_cnn, 0), (tiny_cnn, 1), (tiny_cnn, 2),
    (tiny_resnet, 7), (preact_resnet, 3), (preact_resnet, 0)])
def test_per_sample_replay(make, flags):
    """Recompute every sample's gradient with torch autograd from the logged
    weight versions: forward values from the predicted weights of the forward
    tick, derivatives through the weights current at the backward tick
    (G(x_i; F_i, W_i)); then re-derive every (w, v) version from the update rule."""
    wl = make()
    o = _oracle(wl, record=True, flags=flags)
    S, lr, m = wl.n_stages, wl.lr, wl.momentum
    n = 2 * (S - 1) + 8
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    losses = [o.tick(x[t], y[t]) for t in range(n)]
    stages = torch_ref.build(wl)
    done = sorted({i for (s, i) in o.bwd_version if s == 0})
    assert len(done) >= 8
    for i in done:
        tf, tb = [], []
        for st in stages:
            s = st.index
            D = 2 * (S - 1 - s)
            w, v = o.history[s][o.fwd_version[(s, i)]]
            if flags & 2:
                if flags & 4:
                    wp = o.history[s][max(o.fwd_version[(s, i)] - 1, 0)][0]
                    w_hat = w + D * (w - wp)
                else:
                    w_hat = w - lr * D * v
            else:
                w_hat = w
            tf.append(torch.tensor(w_hat))
            tb.append(torch.tensor(o.history[s][o.bwd_version[(s, i)]][0], requires_grad=True))
        xt = torch.tensor(x[i], dtype=torch.float64).view(*wl.in_shape)
        loss = torch_ref.network_loss(stages, tf, xt, y[i], tb)
        loss.backward()
        assert losses[i + S - 1] == pytest.approx(loss.item(), rel=1e-9)
        for st in stages:
            s = st.index
            g = tb[s].grad.numpy()
            np.testing.assert_allclose(o.grads[(s, i)], g, rtol=1e-8,
                                       atol=1e-10 * max(1.0, np.abs(g).max()))
            # the update that consumed it
            D = 2 * (S - 1 - s)
            a, b = sc_coefficients(m, D) if flags & 1 else (1.0, 0.0)
            w0, v0 = o.history[s][i]
            w1, v1 = o.history[s][i + 1]
            np.testing.assert_allclose(v1, m * v0 + g, rtol=1e-8, atol=1e-10)
            np.testing.assert_allclose(w1, w0 - lr * (a * (m * v0 + g) + b * g), rtol=1e-9, atol=1e-11)


@pytest.mark.parametrize("make,flags", [
    (lambda: mlp([9, 7, 6, 5], lr=0.05), 0), (tiny_cnn, 0), (tiny_resnet, 0),
    (lambda: tiny_resnet(bottleneck=True), 3), (tiny_cnn, 2), (preact_resnet, 3)])
def test_weight_stashing_gives_the_true_gradient_at_the_forward_weights(make, flags):
    """Eq. "W_{i+1} = W_i - eta grad L(x_i; F_i)": with stashing every sample's
    gradient is an ORDINARY backward pass (plain torch autograd, nothing mixed)
    of the network that holds, in stage s, the weights of that sample's forward
    tick; the update then moves the current weights."""
    wl = make()
    o = _oracle(wl, record=True, flags=flags, weight_stash=True)
    S, lr, m = wl.n_stages, wl.lr, wl.momentum
    n = 2 * (S - 1) + 8
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    losses = [o.tick(x[t], y[t]) for t in range(n)]
    stages = torch_ref.build(wl)
    done = sorted({i for (s, i) in o.bwd_version if s == 0})
    assert len(done) >= 8
    differs = False
    for i in done:
        F_i = []
        for st in stages:
            s = st.index
            D = 2 * (S - 1 - s)
            w, v = o.history[s][o.fwd_version[(s, i)]]
            F_i.append(torch.tensor(w - lr * D * v if flags & 2 else w, requires_grad=True))
            differs = differs or o.fwd_version[(s, i)] != o.bwd_version[(s, i)]
        xt = torch.tensor(x[i], dtype=torch.float64).view(*wl.in_shape)
        loss = torch_ref.network_loss(stages, F_i, xt, y[i])
        loss.backward()
        assert losses[i + S - 1] == pytest.approx(loss.item(), rel=1e-9)
        for st in stages:
            s = st.index
            g = F_i[s].grad.numpy()
            np.testing.assert_allclose(o.grads[(s, i)], g, rtol=1e-8, atol=1e-10 * max(1.0, np.abs(g).max()))
            D = 2 * (S - 1 - s)
            a, b = sc_coefficients(m, D) if flags & 1 else (1.0, 0.0)
            w0, v0 = o.history[s][i]
            w1, v1 = o.history[s][i + 1]
            np.testing.assert_allclose(w1, w0 - lr * (a * (m * v0 + g) + b * g), rtol=1e-9, atol=1e-11)
    assert differs                      # forward and backward ticks really saw different weight versions
    # and it is a different trajectory from the one without stashing
    p = _oracle(wl, flags=flags)
    for t in range(n):
        p.tick(x[t], y[t])
    assert not np.allclose(p.get_weights(), o.get_weights(), rtol=1e-6, atol=0)


def test_fill_phase_leaves_state_untouched():
    wl = mlp([6, 5, 4, 3])
    o = _oracle(wl)
    w0 = o.get_weights().copy()
    x, y = make_inputs(wl.seed, 10, 6, 3)
    S = wl.n_stages
    for t in range(S - 1):          # no gradient exists yet anywhere
        o.tick(x[t], y[t])
        np.testing.assert_array_equal(o.get_weights(), w0)
        assert not o.get_velocity().any()
    o.tick(x[S - 1], y[S - 1])      # the last stage updates first (delay 0)
    off = o.n_params - o.stages[-1].n_params
    assert np.array_equal(o.get_weights()[:off], w0[:off])
    assert not np.array_equal(o.get_weights()[off:], w0[off:])


def test_benchmark_networks_have_the_stated_sizes():
    sizes = {"mlp4": (4, 335114), "mlp16x2048": (16, 62965770), "vgg11": (9, 9228362),
             "resnet20": (20, 269722), "resnet50": (54, 25557032)}
    for name, (S, P) in sizes.items():
        wl = workload(name)
        o = PBOracle(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr,
                     wl.momentum, wl.flags)
        assert (o.S, o.n_params) == (S, P)
        assert [o.delay(s) for s in (0, S - 1)] == [2 * (S - 1), 0]


def test_rejects_stage_without_head():
    wl = Workload("bad", [Layer(OP.RELU)], [0], (3, 1, 1), 3, 0.1, 0.9, 1, 0)
    with pytest.raises(Exception):
        PBOracle(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, 0.1, 0.9)


def test_compensation_scales_set_the_stage_constants():
    # SC with alpha*D and horizon alpha*D (SC_2D / LWP_2D are alpha = 2): stage s must use
    # a = m^(alpha_sc D_s), b = (1 - a)/(1 - m), T = alpha_T D_s
    wl = mlp([6, 5, 4, 3])
    o = PBOracle(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, 0.1, 0.9, 3,
                 sc_delay_scale=2, horizon_scale=0.5)
    o.set_weights(he_normal_weights(wl.seed, wl))
    for s, opt in enumerate(o.opt):
        D = 2 * (o.S - 1 - s)
        assert opt.a == pytest.approx(0.9 ** (2 * D), rel=1e-12)
        assert opt.b == pytest.approx((1 - 0.9 ** (2 * D)) / 0.1, rel=1e-12, abs=1e-15)
        assert opt.T == pytest.approx(0.5 * D)
        assert opt.a / 0.1 + opt.b == pytest.approx(10.0, rel=1e-12)     # total contribution unchanged


def test_switching_the_compensation_between_ticks_changes_constants_not_state():
    # Other strengths from some tick on: (w, v) stay as they are, the constants become those
    # of the closed forms, and the very next prediction is w - lr (alpha_T D) v by hand.
    wl = mlp([6, 5, 4, 3], lr=0.05)
    o = _oracle(wl)
    x, y = make_inputs(wl.seed, 12, wl.sample_elems, wl.n_classes)
    for t in range(9):
        o.tick(x[t], y[t])
    w, v = o.get_weights().copy(), o.get_velocity().copy()
    assert v.any()
    o.set_mitigation(2, 0.5)
    np.testing.assert_array_equal(o.get_weights(), w)
    np.testing.assert_array_equal(o.get_velocity(), v)
    for s, opt in enumerate(o.opt):
        D = 2 * (o.S - 1 - s)
        assert opt.a == pytest.approx(0.9 ** (2 * D), rel=1e-12)
        assert opt.b == pytest.approx((1 - 0.9 ** (2 * D)) / 0.1, rel=1e-12, abs=1e-15)
        np.testing.assert_allclose(opt.predicted(), opt.w - 0.05 * (0.5 * D) * opt.v, rtol=1e-14, atol=0)
    # switched at tick 0 it is the same machine as one built with those scales
    a = _oracle(wl); a.set_mitigation(2, 0.5)
    b = _oracle(wl, sc_delay_scale=2, horizon_scale=0.5)
    for t in range(12):
        assert a.tick(x[t], y[t]) == b.tick(x[t], y[t]) or t < o.S - 1
    np.testing.assert_array_equal(a.get_weights(), b.get_weights())


@pytest.mark.parametrize("make,N", [(lambda: mlp([10, 8, 6, 4], lr=0.05), 3), (tiny_cnn, 4),
                                    (tiny_resnet, 2), (lambda: tiny_resnet(bottleneck=True), 5),
                                    (lambda: mlp([9, 5], lr=0.05), 1)])
def test_fill_and_drain_is_minibatch_sgdm(make, N):
    # Filling and draining the pipeline for every update is ordinary mini-batch SGD with
    # momentum (Section 1; Appendix "Pipelined Backpropagation"): torch's SGD on the mean
    # loss of the N samples of a cycle must give the same weights, velocities and losses,
    # and one update must take N + 2S - 2 ticks.
    wl = make()
    S = wl.n_stages
    cycle = N + 2 * S - 2
    o = PBOracle(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum,
                 wl.flags, update_size=N)
    w0 = he_normal_weights(wl.seed, wl).astype(np.float64)
    o.set_weights(w0)
    stages = torch_ref.build(wl)
    params = [torch.nn.Parameter(p) for p in _thetas(stages, w0)]
    ref = torch.optim.SGD(params, lr=wl.lr, momentum=wl.momentum)
    n_cycles = 3
    x, y = make_inputs(wl.seed, n_cycles * cycle, wl.sample_elems, wl.n_classes)
    for c in range(n_cycles):
        base = c * cycle
        w_before = o.get_weights().copy()
        got = [o.tick(x[base + p], y[base + p]) for p in range(cycle)]
        # nothing moved before the pipeline was empty is checked by the cycle's losses:
        # every sample of the cycle saw the weights of the cycle's start
        ref.zero_grad()
        losses = [torch_ref.network_loss(stages, params, torch.tensor(x[base + p], dtype=torch.float64).view(wl.in_shape),
                                         y[base + p]) for p in range(N)]
        (sum(losses) / N).backward()
        for p in range(cycle):
            q = p - (S - 1)              # the sample whose loss appears at tick base + p
            if 0 <= q < N:
                assert got[p] == pytest.approx(losses[q].item(), rel=1e-10, abs=1e-12)
            else:
                assert np.isnan(got[p])
        ref.step()
        want = np.concatenate([p.detach().numpy().ravel() for p in params])
        np.testing.assert_allclose(o.get_weights(), want, rtol=1e-9, atol=1e-12)
        vel = np.concatenate([ref.state[p]["momentum_buffer"].numpy().ravel() for p in params])
        np.testing.assert_allclose(o.get_velocity(), vel, rtol=1e-9, atol=1e-12)
        assert not np.array_equal(o.get_weights(), w_before)


def test_fill_and_drain_holds_the_weights_until_the_pipeline_is_empty():
    wl = mlp([10, 8, 6, 4], lr=0.05)
    N, S = 3, wl.n_stages
    cycle = N + 2 * S - 2
    o = PBOracle(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum,
                 wl.flags, update_size=N)
    w0 = he_normal_weights(wl.seed, wl).astype(np.float64)
    o.set_weights(w0)
    x, y = make_inputs(wl.seed, cycle, wl.sample_elems, wl.n_classes)
    for p in range(cycle - 1):
        o.tick(x[p], y[p])
        np.testing.assert_array_equal(o.get_weights(), w0)
    o.tick(x[cycle - 1], y[cycle - 1])
    assert not np.array_equal(o.get_weights(), w0)
    assert all(op.version == 1 for op in o.opt)
