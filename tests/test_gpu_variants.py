"""Mitigation variants of the paper on the GPU against the CPU checker: the
weight-difference form of LWP (with and without SC), over-compensation
(SC_2D, LWP_2D) and horizons T = alpha D."""
import pytest

from pb_workloads import mlp, tiny_cnn, tiny_resnet, preact_resnet
from tests.parity import compare_ticks

pytestmark = pytest.mark.gpu

TOL = 1e-4


@pytest.mark.parametrize("make", [lambda f: mlp([48, 40, 33, 24, 5], lr=0.003, seed=31, flags=f),
                                  lambda f: tiny_cnn(flags=f), lambda f: _resnet(f)])
@pytest.mark.parametrize("flags", [7, 6])
def test_weight_difference_form(make, flags):
    wl = make(flags)
    n = 2 * (wl.n_stages - 1) + 20
    w = compare_ticks(wl, n, TOL)
    assert w["ticks"] == n


def _resnet(flags):
    wl = tiny_resnet()
    wl.flags = flags
    return wl


@pytest.mark.parametrize("make", [lambda: mlp([48, 40, 33, 24, 5], lr=0.003, seed=32), tiny_cnn])
@pytest.mark.parametrize("scales", [(2.0, 2.0), (2.0, 1.0), (1.0, 2.0), (0.0, 0.5)])
def test_over_and_under_compensation(make, scales):
    wl = make()
    n = 2 * (wl.n_stages - 1) + 20
    w = compare_ticks(wl, n, TOL, mitigation=scales)
    assert w["ticks"] == n


@pytest.mark.parametrize("make", [lambda: mlp([48, 40, 33, 24, 5], lr=0.003, seed=32), tiny_cnn, lambda: _resnet(3)])
def test_compensation_switched_after_every_stage_has_updated(make):
    # conv stages keep their predicted weights in memory: a new horizon must reach them at
    # once (re-made from w and v), as it reaches FC stages, which predict on the fly
    wl = make()
    S = wl.n_stages
    n = 2 * (S - 1) + 24
    w = compare_ticks(wl, n, TOL, mitigation_switch=(2 * (S - 1) + 5, (2.0, 0.5)))
    assert w["ticks"] == n and w["min_updates"] >= 10


def test_weight_difference_form_takes_new_scales_only_before_the_first_tick():
    import torch
    from paper_2003_11666_b200 import PBError
    from pb_workloads import make_inputs
    from tests.parity import make_engine
    wl = tiny_cnn(flags=7)
    e = make_engine(wl)
    e.set_mitigation(2.0, 2.0)                      # tick 0: accepted
    x, y = make_inputs(wl.seed, 2, wl.sample_elems, wl.n_classes)
    e.run(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda(), 2)
    with pytest.raises(PBError) as err:
        e.set_mitigation(1.0, 1.0)
    assert err.value.code == -6
    e.destroy()


def test_mitigation_scale_arguments_are_checked():
    from paper_2003_11666_b200 import PBError
    from tests.parity import make_engine
    e = make_engine(mlp([8, 6, 4]))
    with pytest.raises(PBError):
        e.set_mitigation(-1.0, 1.0)
    e.set_mitigation(1.0, 1.0)
    e.destroy()


def test_wform_needs_lwp():
    from paper_2003_11666_b200 import PB, PBError
    wl = mlp([8, 6, 4])
    with pytest.raises(PBError):
        PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, 0.1, 0.9, flags=4)


def _stashed(wl):
    wl.weight_stash = True
    return wl


@pytest.mark.parametrize("make,tol", [
    (lambda: mlp([48, 40, 33, 24, 5], lr=0.003, seed=33), TOL),
    (lambda: mlp([64, 48, 32, 6], lr=0.003, seed=34, flags=0), TOL),
    (tiny_cnn, TOL), (lambda: tiny_cnn(flags=0), TOL), (lambda: _resnet(3), TOL),
    (lambda: tiny_resnet(bottleneck=True, flags=3), TOL),
    (lambda: tiny_resnet(bottleneck=True, flags=3 | 8, relu=False), 2e-2), (preact_resnet, TOL)])
def test_weight_stashing(make, tol):
    # the comparison mode of the paper's appendix (PipeDream's rule): the backward pass of a
    # sample uses the weights of its own forward pass; FC stages, CUDA-core and tensor-core
    # convolutions, with and without the mitigations
    wl = _stashed(make())
    n = 2 * (wl.n_stages - 1) + 20
    w = compare_ticks(wl, n, tol)
    assert w["ticks"] == n and w["min_updates"] >= 20


def test_weight_stashing_changes_the_trajectory():
    # (so that the test above cannot pass with the flag ignored on both sides)
    import numpy as np
    import torch
    from pb_workloads import make_inputs
    from tests.parity import make_engine
    outs = []
    for stash in (False, True):
        wl = tiny_cnn()
        wl.weight_stash = stash
        e = make_engine(wl)
        n = 2 * (wl.n_stages - 1) + 12
        x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
        e.run(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda(), n)
        e.sync()
        outs.append(e.get_weights())
        e.destroy()
    assert not np.allclose(outs[0], outs[1], rtol=1e-6, atol=0)
