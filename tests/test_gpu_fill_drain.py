"""Fill-and-drain training (mini-batch SGD with momentum on the pipeline,
Section 1 and Appendix "Pipelined Backpropagation") on the GPU against the CPU
checker's fill-and-drain mode, which is itself pinned to torch's SGD.

Losses are compared at every tick (NaN where no sample reaches the last
stage).  Weights and velocities are compared at the end of every cycle of
N + 2S - 2 ticks: inside a cycle the engine lets a stage step as soon as its own
last backward of the cycle is done, the checker when the pipeline is empty;
both hold the same state whenever a cycle ends."""
import math

import numpy as np
import pytest

from pb_workloads import make_inputs, mlp, tail_cnn, tiny_cnn, tiny_resnet, preact_resnet
from tests.parity import make_engine, make_oracle, rel_err

pytestmark = pytest.mark.gpu

TOL = 1e-4


def _bottleneck_bf16():
    return tiny_resnet(bottleneck=True, flags=3 | 8)


def _run(wl, N, n_cycles, tol, tol_v=None, use_run=False):
    import torch
    S = wl.n_stages
    cycle = N + 2 * S - 2
    n = n_cycles * cycle
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    o = make_oracle(wl, update_size=N)
    eng = make_engine(wl)
    eng.set_update_size(N)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    worst = 0.0
    for c in range(n_cycles):
        w_start = eng.get_weights()
        if use_run:
            ld = torch.zeros(cycle, device="cuda")
            eng.run(xd[c * cycle:(c + 1) * cycle], yd[c * cycle:(c + 1) * cycle], cycle, ld)
            eng.sync()
            got = ld.cpu().numpy()
        else:
            got = []
            for p in range(cycle):
                t = c * cycle + p
                got.append(eng.tick(xd[t], int(y[t])))
        for p in range(cycle):
            t = c * cycle + p
            lo = o.tick(x[t], y[t])
            if math.isnan(lo):
                assert math.isnan(got[p]), "tick %d: loss should be NaN (no sample at the last stage)" % t
            else:
                e = abs(got[p] - lo) / max(abs(lo), float(np.abs(o.last_logits).max()), 1e-12)
                worst = max(worst, e)
                assert e <= tol, "tick %d: loss %r vs %r" % (t, got[p], lo)
        ew = rel_err(eng.get_weights(), o.get_weights())
        ev = rel_err(eng.get_velocity(), o.get_velocity())
        assert ew <= tol, "cycle %d: weights rel err %.3g" % (c, ew)
        assert ev <= (tol_v or tol), "cycle %d: velocity rel err %.3g" % (c, ev)
        assert not np.array_equal(eng.get_weights(), w_start)
    eng.destroy()
    return worst


@pytest.mark.parametrize("make,N", [(lambda: mlp([48, 40, 33, 24, 5], lr=0.02, seed=41), 4),
                                    (lambda: mlp([48, 40, 33, 24, 5], lr=0.02, seed=42), 1),
                                    (lambda: mlp([2048, 300, 10], lr=0.01, seed=43), 3),
                                    (tiny_cnn, 5), (tiny_resnet, 3), (tail_cnn, 4),
                                    (lambda: tiny_resnet(bottleneck=True), 4), (preact_resnet, 3)])
def test_fill_and_drain_matches_minibatch_sgdm(make, N):
    _run(make(), N, 4, TOL)


def test_fill_and_drain_through_pb_run():
    _run(mlp([64, 48, 32, 6], lr=0.02, seed=44), 6, 3, TOL, use_run=True)
    _run(tiny_cnn(), 3, 3, TOL, use_run=True)


def test_fill_and_drain_bf16_convolutions():
    # operands rounded to bfloat16 on both sides; float32-level differences can flip a
    # rounding, so velocities get the bf16 path's looser bound
    _run(_bottleneck_bf16(), 3, 3, 2e-2, tol_v=6e-2)


def test_weights_hold_still_until_the_last_sample_returns():
    import torch
    wl = mlp([32, 24, 16, 4], lr=0.05, seed=45)
    N, S = 4, wl.n_stages
    cycle = N + 2 * S - 2
    x, y = make_inputs(wl.seed, cycle, wl.sample_elems, wl.n_classes)
    eng = make_engine(wl)
    eng.set_update_size(N)
    w0 = eng.get_weights()
    xd = torch.from_numpy(x).cuda()
    # the last stage sees the last sample's gradient at tick N-1 + S-1; before that
    # no weight anywhere may change
    for t in range(N - 1 + S - 1):
        eng.tick(xd[t], int(y[t]))
        np.testing.assert_array_equal(eng.get_weights(), w0)
    for t in range(N - 1 + S - 1, cycle):
        eng.tick(xd[t], int(y[t]))
    assert (eng.get_weights() != w0).mean() > 0.5
    eng.destroy()


def test_update_size_must_be_set_before_the_first_tick():
    import torch
    from paper_2003_11666_b200 import PBError
    wl = mlp([8, 6, 4])
    eng = make_engine(wl)
    with pytest.raises(PBError):
        eng.set_update_size(-1)
    eng.set_update_size(2)
    eng.set_update_size(0)
    x, y = make_inputs(wl.seed, 1, wl.sample_elems, wl.n_classes)
    eng.tick(torch.from_numpy(x).cuda()[0], int(y[0]))
    with pytest.raises(PBError):
        eng.set_update_size(2)
    eng.destroy()
