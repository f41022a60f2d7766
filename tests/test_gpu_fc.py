"""CUDA engine vs CPU checker on fully connected pipelines (through the C ABI)."""
import numpy as np
import pytest

from pb_workloads import mlp, workload, make_inputs, he_normal_weights
from tests.parity import compare_ticks, make_engine, make_oracle, rel_err

pytestmark = pytest.mark.gpu

TOL = 1e-4      # relative, float32 path


@pytest.mark.parametrize("sizes", [[12, 7], [20, 16, 5], [33, 17, 9, 4], [784, 256, 256, 256, 10],
                                   [130, 260, 131, 70, 3], [512, 300, 10]])
@pytest.mark.parametrize("flags", [3, 0, 1, 2])
def test_small_mlps_match_checker(sizes, flags):
    # odd widths reach the scalar path, ragged chunks and rows that are not a multiple of 4
    wl = mlp(sizes, lr=0.002, seed=21, flags=flags)
    S = wl.n_stages
    w = compare_ticks(wl, 2 * (S - 1) + 24, TOL)
    assert w["ticks"] == 2 * (S - 1) + 24


def test_mlp4_first_64_ticks():
    # literal benchmark hyper-parameters; these dynamics are diverging, and from
    # tick ~54 on even float32 evaluation of the checker itself drifts past 1e-4
    # from float64, so the strict bound is held on ticks < 40 and a 2e-3 bound after.
    wl = workload("mlp4")
    w = compare_ticks(wl, 64, TOL, loose_after=(40, 2e-3))
    assert w["ticks"] == 64


def test_mlp4_stable_learning_rate_64_ticks():
    wl = workload("mlp4")
    wl.lr = 0.001
    w = compare_ticks(wl, 64, TOL)
    assert w["ticks"] == 64


def test_deep_mlp_full_size_until_float32_range_ends():
    # Full benchmark size (63 M parameters, 16 stages), literal hyper-parameters.
    # lr*|x|^2 is about 10 here, so the run diverges: the checker's weights pass
    # 1e30 near tick 34, where float32 overflows; the comparison covers every tick
    # up to there (all 16 stages have updated by tick 30).  The weights are compared
    # on every third tick to keep the float64 norms affordable.
    # Per tensor the strict bound holds through tick 30, when the first stage takes its first
    # update; in the last three ticks before the overflow every quantity grows a thousandfold
    # per tick and rounding differences with it (2e-3 there, as for the 4-stage MLP).
    wl = workload("mlp16x2048")
    w = compare_ticks(wl, 64, TOL, check_every=3, finite_limit=1e24, loose_after=(31, 2e-3))
    assert 31 <= w["ticks"] <= 36, w


def test_deep_mlp_narrow_stable_64_ticks():
    # same depth (16 stages, delays 30..0) at width 256 with a stable step: all 64 ticks
    wl = mlp([256] * 16 + [10], lr=0.0005, seed=1)
    w = compare_ticks(wl, 2 * 15 + 34, TOL)
    assert w["ticks"] == 64


def test_run_matches_tick_by_tick_and_loss_is_delayed():
    import torch
    wl = mlp([64, 48, 32, 6], lr=0.003, seed=5)
    n = 40
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    a, b = make_engine(wl), make_engine(wl)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    losses = torch.zeros(n, device="cuda")
    a.run(xd, yd, n, losses)
    a.sync()
    one = [b.tick(xd[t], int(y[t])) for t in range(n)]
    got = losses.cpu().numpy()
    S = wl.n_stages
    assert np.isnan(got[:S - 1]).all() and np.isfinite(got[S - 1:]).all()
    np.testing.assert_array_equal(got[S - 1:], np.array(one[S - 1:], dtype=np.float32))
    np.testing.assert_array_equal(a.get_weights(), b.get_weights())
    assert a.tick_count == n and a.last_launch_count == n      # one launch per tick
    # host-buffer entry point gives the same numbers
    c = make_engine(wl)
    hl = np.zeros(n, dtype=np.float32)
    c.run_host(x, y, n, hl)
    np.testing.assert_array_equal(hl[S - 1:], got[S - 1:])
    np.testing.assert_array_equal(c.get_weights(), a.get_weights())
    for e in (a, b, c):
        e.destroy()


def test_set_weights_restarts_the_pipeline():
    import torch
    wl = mlp([32, 16, 4], lr=0.01, seed=6)
    x, y = make_inputs(wl.seed, 12, wl.sample_elems, wl.n_classes)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    e = make_engine(wl)
    l1 = torch.zeros(12, device="cuda")
    e.run(xd, yd, 12, l1)
    w1 = e.get_weights()
    e.set_weights(he_normal_weights(wl.seed, wl))
    assert e.tick_count == 0 and not e.get_velocity().any()
    l2 = torch.zeros(12, device="cuda")
    e.run(xd, yd, 12, l2)
    np.testing.assert_array_equal(w1, e.get_weights())
    np.testing.assert_array_equal(l1.cpu().numpy()[2:], l2.cpu().numpy()[2:])
    e.destroy()


def test_bad_arguments_are_reported_not_thrown_across_the_abi():
    from paper_2003_11666_b200 import PB, PBError
    wl = mlp([8, 4])
    with pytest.raises(PBError):
        PB(wl.layers, wl.stage_of_layer, (9, 1, 1), 4, 0.1, 0.9)      # FC size mismatch
    with pytest.raises(PBError):
        PB(wl.layers, wl.stage_of_layer, wl.in_shape, 4, 0.1, 1.5)    # momentum out of range
    e = make_engine(wl)
    with pytest.raises(PBError):
        e.set_weights(np.zeros(3, np.float32))
    with pytest.raises(PBError):
        e.tick(0, 99)
    e.destroy()


def test_misaligned_sample_buffer_is_rejected_on_the_host():
    # the first FC stage reads the caller's sample 16 bytes at a time when its length is a
    # multiple of 4: a float pointer that is only 4-byte aligned must come back as PB_E_ARG
    # from the host-side check (nothing is launched), not as a device fault
    import torch
    from paper_2003_11666_b200 import PBError
    wl = mlp([64, 16, 4], lr=0.01, seed=6)
    e = make_engine(wl)
    buf = torch.zeros(4 * 64 + 8, device="cuda")
    lab = torch.zeros(4, dtype=torch.int32, device="cuda")
    before = e.tick_count
    for call in (lambda p: e.tick(p, 0, want_loss=False), lambda p: e.run(p, lab, 2)):
        with pytest.raises(PBError) as err:
            call(buf.data_ptr() + 4)
        assert err.value.code == -1 and "aligned" in str(err.value)
    assert e.tick_count == before
    e.run(buf, lab, 2)                               # the aligned buffer is fine
    e.sync()
    # a sample length that is not a multiple of 4 takes the scalar path: any float pointer will do
    wl2 = mlp([30, 8, 3], lr=0.01, seed=6)
    e2 = make_engine(wl2)
    e2.run(buf.data_ptr() + 4, lab, 2)
    e2.sync()
    e.destroy(); e2.destroy()


def test_single_stage_network_on_the_gpu():
    # S = 1: delay 0, the sample and its label are consumed in the tick that ingests them
    wl = mlp([40, 6], lr=0.01, seed=8)
    w = compare_ticks(wl, 20, TOL)
    assert w["ticks"] == 20


def test_last_stage_too_large_to_fuse_uses_its_own_launch():
    # 300 outputs (> 256 rows): the loss/backward of the last stage is a second launch
    import torch
    wl = mlp([96, 64, 300], lr=0.002, seed=9)
    w = compare_ticks(wl, 2 * (wl.n_stages - 1) + 16, TOL)
    assert w["ticks"] == 2 * (wl.n_stages - 1) + 16
    e = make_engine(wl)
    x, y = make_inputs(wl.seed, 4, wl.sample_elems, wl.n_classes)
    e.run(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda(), 4)
    e.sync()
    assert e.last_launch_count == 8
    e.destroy()


def test_long_run_equals_single_ticks_bit_for_bit():
    # 203 ticks through pb_run (no host involvement between ticks) against 203 pb_tick calls,
    # with the mitigations on and in fill-and-drain mode: losses (NaN positions included),
    # weights and velocities must be identical
    import torch
    for update_size in (0, 5):
        wl = mlp([96, 80, 64, 48, 7], lr=0.002, seed=12)
        n = 203
        x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
        xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
        a, b = make_engine(wl), make_engine(wl)
        if update_size:
            a.set_update_size(update_size); b.set_update_size(update_size)
        la = torch.zeros(n, device="cuda")
        a.run(xd, yd, n, la)
        a.sync()
        one = np.array([b.tick(xd[t], int(y[t])) for t in range(n)], dtype=np.float32)
        np.testing.assert_array_equal(la.cpu().numpy(), one)
        np.testing.assert_array_equal(a.get_weights(), b.get_weights())
        np.testing.assert_array_equal(a.get_velocity(), b.get_velocity())
        a.destroy(); b.destroy()


def test_consecutive_runs_and_ticks_form_one_stream_and_zero_ticks_is_a_no_op():
    import torch
    wl = mlp([48, 40, 24, 5], lr=0.003, seed=10)
    n = 30
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    xd, yd = torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()
    a, b = make_engine(wl), make_engine(wl)
    la = torch.zeros(n, device="cuda")
    a.run(xd, yd, n, la)
    lb = torch.zeros(n, device="cuda")
    b.run(xd[:7], yd[:7], 7, lb[:7])
    b.run(xd[7:7], yd[7:7], 0, None)                       # nothing happens
    one = b.tick(xd[7], int(y[7]))                           # odd tick count in between
    b.run(xd[8:], yd[8:], n - 8, lb[8:])
    a.sync(); b.sync()
    S = wl.n_stages
    got_a, got_b = la.cpu().numpy(), lb.cpu().numpy()
    got_b[7] = one
    np.testing.assert_array_equal(got_a[S - 1:], got_b[S - 1:])
    np.testing.assert_array_equal(a.get_weights(), b.get_weights())
    np.testing.assert_array_equal(a.get_velocity(), b.get_velocity())
    assert b.tick_count == n
    a.destroy(); b.destroy()
