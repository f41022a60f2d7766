"""The comparison the GPU parity tests use must be able to fail: it is fed the
CPU checker's own state with ONE stage's latest update redone with a wrong
spike-compensation coefficient (host arithmetic only) and has to reject it at
the loosest tolerance any GPU test uses (2e-2, the bfloat16 path), while a
single norm over all parameters would have let it through."""
import numpy as np

from pb_workloads import he_normal_weights, make_inputs, tiny_resnet
from tests.parity import compare_state, make_oracle, rel_err, tensor_slices, update_rule_residual

TOL_BF16 = 2e-2


def _run(n_ticks):
    wl = tiny_resnet(bottleneck=True, flags=3)
    o = make_oracle(wl, record=True)
    x, y = make_inputs(wl.seed, n_ticks, wl.sample_elems, wl.n_classes)
    for t in range(n_ticks):
        o.tick(x[t], y[t])
    return wl, o


def _stage_offset(o, s):
    return sum(st.n_params for st in o.stages[:s])


def test_a_wrong_spike_coefficient_in_one_stage_is_rejected():
    S = 13
    wl, o = _run(2 * (S - 1) + 6)
    assert o.S == S
    slices = tensor_slices(o)
    w_init = he_normal_weights(wl.seed, wl)
    ref_w, ref_v = o.get_weights(), o.get_velocity()
    updates = [op.version for op in o.opt]
    assert min(updates) >= 1
    # the checker's own state passes
    rw, rv, fails = compare_state(slices, w_init, ref_w.astype(np.float32), ref_v.astype(np.float32),
                                  ref_w, ref_v, updates, TOL_BF16, TOL_BF16)
    assert not fails and rw < 1e-2 and rv < 1e-2
    for s in (0, 3, S - 1):
        op = o.opt[s]
        (w_prev, v_prev), (w_now, v_now) = o.history[s][-2], o.history[s][-1]
        g = v_now - op.m * v_prev                       # the gradient of the latest update
        # plain momentum step (b = 0) where SC_D asks for b = (1 - m^D)/(1 - m):
        # the mistake a kernel makes that drops the spike term
        wrong_b = 0.0 if op.b != 0 else 1.0
        w_bad = w_prev - op.lr * (op.a * v_now + wrong_b * g)
        got_w = ref_w.copy()
        off = _stage_offset(o, s)
        got_w[off:off + w_bad.size] = w_bad
        rw, rv, fails = compare_state(slices, w_init, got_w, ref_v, ref_w, ref_v, updates, TOL_BF16, TOL_BF16)
        assert fails and rw > 1.0, "stage %d: a dropped spike term went unnoticed" % s
        assert all(("stage %d " % s) in f for f in fails)
    # ... while one norm over the whole parameter vector does not see the last stage's mistake
    s = S - 1
    op = o.opt[s]
    (w_prev, v_prev), (w_now, v_now) = o.history[s][-2], o.history[s][-1]
    g = v_now - op.m * v_prev
    got_w = ref_w.copy()
    off = _stage_offset(o, s)
    got_w[off:] = w_prev - op.lr * (op.a * v_now + 1.0 * g)
    assert rel_err(got_w, ref_w) < TOL_BF16


def test_a_ten_percent_error_in_b_is_rejected_in_a_late_and_an_early_stage():
    S = 13
    wl, o = _run(2 * (S - 1) + 6)
    slices = tensor_slices(o)
    w_init = he_normal_weights(wl.seed, wl)
    ref_w, ref_v = o.get_weights(), o.get_velocity()
    updates = [op.version for op in o.opt]
    for s in (0, 5):
        op = o.opt[s]
        # redo EVERY update of the stage with b 10 % too small (the same gradients)
        w = o.history[s][0][0].copy()
        for q in range(1, len(o.history[s])):
            v_prev, v_now = o.history[s][q - 1][1], o.history[s][q][1]
            g = v_now - op.m * v_prev
            w = w - op.lr * (op.a * v_now + 0.9 * op.b * g)
        got_w = ref_w.copy()
        off = _stage_offset(o, s)
        got_w[off:off + w.size] = w
        _, _, fails = compare_state(slices, w_init, got_w, ref_v, ref_w, ref_v, updates, TOL_BF16, TOL_BF16)
        assert fails, "stage %d" % s


def test_state_that_must_not_move_is_held_to_its_bits():
    S = 13
    wl, o = _run(S + 3)                # the last stages have updated, the first ones not yet
    slices = tensor_slices(o)
    w_init = he_normal_weights(wl.seed, wl)
    ref_w, ref_v = o.get_weights(), o.get_velocity()
    updates = [op.version for op in o.opt]
    assert updates[0] == 0 and updates[-1] > 0
    ok = compare_state(slices, w_init, ref_w.astype(np.float32), ref_v.astype(np.float32), ref_w, ref_v,
                       updates, 1e-4, 1e-4)
    assert not ok[2]
    got_v = ref_v.copy()
    got_v[3] = 1e-30                   # a velocity of stage 0 that is not exactly zero
    assert compare_state(slices, w_init, ref_w, got_v, ref_w, ref_v, updates, 1e-4, 1e-4)[2]
    got_w = ref_w.astype(np.float32)
    got_w[5] = np.nextafter(got_w[5], np.float32(np.inf))     # one ulp on a weight nobody has updated
    assert compare_state(slices, w_init, got_w, ref_v, ref_w, ref_v, updates, 1e-4, 1e-4)[2]


def test_float32_rounding_of_the_weights_alone_passes_the_strict_tolerance():
    # the engine keeps w in float32: storing the checker's float64 state in float32 after a
    # few small updates must not trip the 1e-4 displacement bound (rounding floor)
    S = 13
    wl, o = _run(2 * (S - 1) + 12)
    slices = tensor_slices(o)
    w_init = he_normal_weights(wl.seed, wl)
    ref_w, ref_v = o.get_weights(), o.get_velocity()
    updates = [op.version for op in o.opt]
    _, _, fails = compare_state(slices, w_init, ref_w.astype(np.float32), ref_v.astype(np.float32), ref_w, ref_v,
                                updates, 1e-4, 1e-4)
    assert not fails


def test_update_rule_property_accepts_the_checker_and_rejects_a_wrong_coefficient():
    # the property the GPU tests check on the engine's own consecutive states: fed the
    # checker's states (rounded to float32, as the engine stores them) it holds; with one
    # stage's step redone with b 10 % off, or with the SC term dropped, it does not
    S = 13
    wl = tiny_resnet(bottleneck=True, flags=3)
    o = make_oracle(wl, record=True)
    n = 2 * (S - 1) + 8
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    for t in range(n - 1):
        o.tick(x[t], y[t])
    w0, v0 = o.get_weights().astype(np.float32), o.get_velocity().astype(np.float32)
    o.tick(x[n - 1], y[n - 1])
    w1, v1 = o.get_weights().astype(np.float32), o.get_velocity().astype(np.float32)
    slices = tensor_slices(o)
    assert update_rule_residual(o, slices, w0, v0, w1, v1) <= 1.0
    for s, scale in ((0, 0.9), (4, 0.9), (7, 0.0)):
        op = o.opt[s]
        off = _stage_offset(o, s)
        sl = slice(off, off + op.w.size)
        g = v1[sl].astype(np.float64) - float(op.m) * v0[sl]
        bad = w1.copy()
        bad[sl] = (w0[sl] - float(op.lr) * (float(op.a) * v1[sl] + scale * float(op.b) * g)).astype(np.float32)
        assert update_rule_residual(o, slices, w0, v0, bad, v1) > 1.0, "stage %d" % s


def test_checker_in_its_own_process_gives_the_same_numbers():
    # the full-size GPU comparisons run the checker in spawned processes; same bits as in-process
    from tests.oracle_proc import RemoteOracle
    wl = tiny_resnet()
    n = 2 * (wl.n_stages - 1) + 3
    x, y = make_inputs(wl.seed, n, wl.sample_elems, wl.n_classes)
    o = make_oracle(wl)
    r = RemoteOracle(wl)
    try:
        for t in range(n):
            r.tick_begin(x[t], y[t])
            lo = o.tick(x[t], y[t])
            lr_ = r.tick_end()
            assert (np.isnan(lo) and np.isnan(lr_)) or lo == lr_
        w, v, ver = r.state()
        np.testing.assert_array_equal(w, o.get_weights())
        np.testing.assert_array_equal(v, o.get_velocity())
        assert ver == [p.version for p in o.opt]
    finally:
        r.close()
