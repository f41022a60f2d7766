"""Shared helpers of the GPU parity tests: run the CUDA engine and the CPU
checker on the same seeded inputs and compare per tick, per stage and per
parameter tensor."""
import math

import numpy as np

from oracle import PBOracle
from pb_workloads import he_normal_weights, make_inputs

F32_HALF_ULP = 2.0 ** -24      # relative rounding error of one float32 store


def rel_err(got, ref):
    """||got - ref||_2 / max(||ref||_2, 1e-12); tensors that are exactly zero
    in the reference must be exactly zero."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    n = np.linalg.norm(ref)
    if n == 0.0:
        return 0.0 if not got.any() else float("inf")
    return float(np.linalg.norm(got - ref) / max(n, 1e-12))


def tensor_slices(o):
    """[(stage, kind, slice)] of every parameter tensor in the flat vector the
    checker `o` (and the engine) use: FC weight / bias, conv weight / GroupNorm
    scale / shift, in layer order."""
    out, off = [], 0
    for st in o.stages:
        h = st.head
        if int(h.op) == 0:                      # FC
            nw = h.c_in * h.c_out
            out.append((st.index, "weight", slice(off, off + nw)))
            out.append((st.index, "bias", slice(off + nw, off + nw + h.c_out)))
        else:
            nw = h.c_out * h.c_in * h.k * h.k
            out.append((st.index, "weight", slice(off, off + nw)))
            if st.gn_groups:
                out.append((st.index, "gamma", slice(off + nw, off + nw + h.c_out)))
                out.append((st.index, "beta", slice(off + nw + h.c_out, off + nw + 2 * h.c_out)))
        off += st.n_params
    assert off == o.n_params
    return out


def compare_state(slices, w_init, got_w, got_v, ref_w, ref_v, updates, tol_w, tol_v):
    """Per-tensor comparison of one tick's state.  Pure numpy (no GPU).

    For every parameter tensor:
      * velocity: ||got_v - ref_v|| <= tol_v * ||ref_v||; a velocity that is
        exactly zero in the reference (no gradient has reached the stage yet,
        Appendix "Pipelined Backpropagation", Eq. F_i) must be exactly zero;
      * weights, through their DISPLACEMENT from the initial values, so that a
        wrong update cannot hide behind the unchanged bulk of the weights:
        ||got_w - ref_w|| <= tol_w * ||ref_w - w_init|| + floor, where floor =
        2^-24 sqrt(n) ||ref_w|| is the rounding of n float32 stores of w
        (n = updates of that stage so far); weights that have not moved in the
        reference must still hold their initial bits.
    tol_w / tol_v: a number, or a dict {(stage, kind): number}.
    Returns (worst weight ratio, worst velocity ratio, failures): ratios are
    error / allowed (<= 1 passes), failures a list of messages."""
    worst_w = worst_v = 0.0
    fails = []
    for s, kind, sl in slices:
        tw = tol_w[(s, kind)] if isinstance(tol_w, dict) else tol_w
        tv = tol_v[(s, kind)] if isinstance(tol_v, dict) else tol_v
        rw = np.asarray(ref_w[sl], np.float64)
        rv = np.asarray(ref_v[sl], np.float64)
        gw = np.asarray(got_w[sl], np.float64)
        gv = np.asarray(got_v[sl], np.float64)
        w0 = np.asarray(w_init[sl], np.float64)
        # velocity
        nv = np.linalg.norm(rv)
        if nv == 0.0:
            if gv.any():
                fails.append("stage %d %s: velocity must be exactly zero before the stage's first gradient" % (s, kind))
                worst_v = float("inf")
        else:
            r = float(np.linalg.norm(gv - rv) / (tv * nv))
            worst_v = max(worst_v, r)
            if not r <= 1.0:
                fails.append("stage %d %s: velocity rel err %.3g (bound %.3g)" % (s, kind, r * tv, tv))
        # weights
        nd = np.linalg.norm(rw - w0)
        if nd == 0.0:
            if not np.array_equal(np.asarray(got_w[sl], np.float32), np.asarray(w_init[sl], np.float32)):
                fails.append("stage %d %s: weights moved although the reference has not updated them" % (s, kind))
                worst_w = float("inf")
        else:
            n_upd = updates[s] if updates is not None else 1
            allowed = tw * nd + F32_HALF_ULP * math.sqrt(max(n_upd, 1)) * np.linalg.norm(rw)
            r = float(np.linalg.norm(gw - rw) / allowed)
            worst_w = max(worst_w, r)
            if not r <= 1.0:
                fails.append("stage %d %s: weight displacement rel err %.3g (bound %.3g)"
                             % (s, kind, float(np.linalg.norm(gw - rw) / nd), tw))
    return worst_w, worst_v, fails


def update_rule_residual(o, slices, w_before, v_before, w_after, v_after, rel=2e-3):
    """A property of every correct tick, checked on the engine's own states of
    two consecutive ticks (no trajectory comparison, so it stays sharp where
    gradients of two correct evaluations differ): with g = v' - m v, the
    gradient the stage must have used, the weights have to satisfy the
    combined-mitigation step w' = w - lr (a_s v' + b_s g) with the stage's SC_D
    coefficients (a = m^D, b = (1 - m^D)/(1 - m) from the checker's
    `sc_coefficients`, D_s = 2 (S - 1 - s)).  Returns the largest
    ||w' - expected|| / (rel * ||step|| + 2^-22 ||w||) over all tensors; <= 1
    passes (rel covers the float32 rounding of the step itself)."""
    worst = 0.0
    for s, kind, sl in slices:
        op = o.opt[s]
        m, lr, a, b = float(op.m), float(op.lr), float(op.a), float(op.b)
        v0, v1 = np.asarray(v_before[sl], np.float64), np.asarray(v_after[sl], np.float64)
        w0, w1 = np.asarray(w_before[sl], np.float64), np.asarray(w_after[sl], np.float64)
        g = v1 - m * v0
        step = -lr * (a * v1 + b * g)
        if not v1.any() and not v0.any():
            continue
        allowed = rel * np.linalg.norm(step) + 4 * F32_HALF_ULP * np.linalg.norm(w1) \
            + lr * (a + b) * 4 * F32_HALF_ULP * (np.linalg.norm(v1) + m * np.linalg.norm(v0))
        worst = max(worst, float(np.linalg.norm(w1 - (w0 + step)) / max(allowed, 1e-300)))
    return worst


def tensor_spread(slices, a_w, a_v, b_w, b_v, w_init):
    """Per-tensor distance between two runs of the checker (float32 and
    float64): {(stage, kind): (weight displacement spread, velocity spread)}."""
    out = {}
    for s, kind, sl in slices:
        nd = np.linalg.norm(np.asarray(b_w[sl], np.float64) - np.asarray(w_init[sl], np.float64))
        nv = np.linalg.norm(np.asarray(b_v[sl], np.float64))
        dw = np.linalg.norm(np.asarray(a_w[sl], np.float64) - np.asarray(b_w[sl], np.float64))
        dv = np.linalg.norm(np.asarray(a_v[sl], np.float64) - np.asarray(b_v[sl], np.float64))
        out[(s, kind)] = (float(dw / nd) if nd > 0 else 0.0, float(dv / nv) if nv > 0 else 0.0)
    return out


def make_oracle(wl, dtype=np.float64, **kw):
    if wl.flags & 8:
        kw.setdefault("conv_operands", "bf16")
    if getattr(wl, "weight_stash", False):
        kw.setdefault("weight_stash", True)
    o = PBOracle(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum,
                 wl.flags & 7, dtype=dtype, **kw)
    o.set_weights(he_normal_weights(wl.seed, wl))
    return o


def make_engine(wl):
    import torch
    from paper_2003_11666_b200 import PB
    flags = wl.flags | (16 if getattr(wl, "weight_stash", False) else 0)
    eng = PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum,
             flags, stream=torch.cuda.current_stream().cuda_stream)
    eng.set_weights(he_normal_weights(wl.seed, wl))
    return eng


class _LocalOracle:
    """The checker in this process, behind the calls `tests/oracle_proc.RemoteOracle` has."""

    def __init__(self, wl, dtype=np.float64, **kw):
        self.o = make_oracle(wl, dtype=dtype, **kw)
        self.last_max_logit = 0.0

    def tick_begin(self, x, y):
        self._args = (x, y)

    def tick_end(self):
        loss = self.o.tick(*self._args)
        if self.o.last_logits is not None:
            self.last_max_logit = float(np.abs(self.o.last_logits).max())
        return loss

    def state(self):
        return self.o.get_weights(), self.o.get_velocity(), [p.version for p in self.o.opt]

    def set_mitigation(self, *scales):
        self.o.set_mitigation(*scales)

    def close(self):
        pass


def compare_ticks(wl, n_ticks, tol, check_every=1, finite_limit=1e30, loose_after=None,
                  fragile_margin=None, fragile_tol=None, spread_factor=None, mitigation=None,
                  plain_loss_tol=None, unrounded_loss_tol=None, check_ticks=None, mitigation_switch=None,
                  flip_allowance=None, check_update_rule=False, parallel=False):
    """Tick both sides one sample at a time; returns the worst errors seen.

    Weights and velocities are compared per stage and per tensor
    (`compare_state`); `worst["w"]`, `worst["v"]` are the largest error /
    allowed ratios times the tolerance (so they read as relative errors).

    The window ends early (returning the tick) once the checker's own state
    exceeds `finite_limit`: past that the float32 engine is out of range.

    fragile_margin / fragile_tol: a ReLU or max-pool decision is an integer
    taken from a floating-point number; when the checker sees one that is
    closer to flipping than `fragile_margin` (relative to the tensor's rms),
    either outcome is a valid float32 result and the two sides may part by a
    finite step.  The strict tolerance holds until the first such decision
    reaches its backward pass; from that tick on `fragile_tol` bounds the
    distance instead.

    spread_factor: for arithmetic that amplifies rounding-order differences
    (bfloat16 operands: a float32-level change can flip a bfloat16 rounding,
    which moves ReLU decisions), the checker is also run in float32 and the
    bound on a STAGE's tensors at a tick becomes max(tol, spread_factor * the
    largest distance between the float32 and float64 runs over the tensors of
    that stage and of the stages after it, whose gradients feed it).

    plain_loss_tol: also bound the plain ratio |dl| / |l| on ticks where the
    loss is not small against the logits (l > 1e-3 max|logit|).
    unrounded_loss_tol: also run the checker WITHOUT operand rounding (the
    paper's arithmetic in float64) and bound the engine's loss against it.
    check_ticks: explicit set of ticks at which the state is compared.
    mitigation_switch: (tick, (SC delay scale, horizon scale)): both sides
    change their compensation strengths before that tick.
    flip_allowance: c.  With bfloat16 operands a ReLU decision can come out
    either way on two correct evaluations; one flipped unit moves a sample's
    gradient by about 1/sqrt(N) of its norm, N the number of units of that
    activation.  The bound of every tensor is then at least c/sqrt(N_min),
    N_min the smallest ReLU'd activation after the first stage (whose inputs
    are identical on both sides); nothing is added for networks without such
    decisions.
    parallel: run every instance of the checker in a process of its own, side by
    side with the engine (full-size networks; not with fragile_margin).
    check_update_rule: at consecutive compared ticks also check the ENGINE'S OWN
    step against the paper's update rule (see `update_rule_residual`)."""
    import torch
    x, y = make_inputs(wl.seed, n_ticks, wl.sample_elems, wl.n_classes)
    okw = {}
    if mitigation is not None:       # (SC delay scale, LWP horizon scale), e.g. (2, 2) for SC_2D + LWP_2D
        okw = dict(sc_delay_scale=mitigation[0], horizon_scale=mitigation[1])
    assert not (parallel and fragile_margin is not None)
    if parallel:
        from tests.oracle_proc import RemoteOracle as Side
    else:
        Side = _LocalOracle
    # `meta` is never ticked in parallel mode: it gives the stage list, the tensor layout and the
    # per-stage constants; in local mode it is the float64 checker itself
    main = Side(wl, margins=fragile_margin is not None, **okw)
    meta = main.o if not parallel else make_oracle(wl, **okw)
    side32 = Side(wl, dtype=np.float32, **okw) if spread_factor is not None else None
    sideplain = Side(wl, conv_operands=None, **okw) if unrounded_loss_tol is not None else None
    sides = [q for q in (main, side32, sideplain) if q is not None]
    fragile_tick = None
    slices = tensor_slices(meta)
    S_ = meta.S
    w_init = he_normal_weights(wl.seed, wl)
    eng = make_engine(wl)
    if mitigation is not None:
        eng.set_mitigation(*mitigation)
    xd = torch.from_numpy(x).cuda()
    flip_floor = np.zeros(S_)
    if flip_allowance is not None:
        sizes = [float(np.prod(st.z_shape)) for st in meta.stages if st.relu and st.index > 0]
        if sizes:
            flip_floor[:] = flip_allowance / math.sqrt(min(sizes))
    prev_state = None
    loss_spread = plain_spread = 0.0
    worst = {"loss": 0.0, "w": 0.0, "v": 0.0, "ticks": 0, "update_rule": 0.0,
             "fragile_tick": None, "strict_w": 0.0, "strict_v": 0.0,
             "plain_loss": 0.0, "unrounded_loss": 0.0, "min_updates": 0}
    try:
        for t in range(n_ticks):
            if mitigation_switch is not None and t == mitigation_switch[0]:
                for q in sides:
                    q.set_mitigation(*mitigation_switch[1])
                if parallel:
                    meta.set_mitigation(*mitigation_switch[1])
                eng.set_mitigation(*mitigation_switch[1])
            for q in sides:
                q.tick_begin(x[t], y[t])
            lg = eng.tick(xd[t], int(y[t]))
            lo = main.tick_end()
            lo32 = side32.tick_end() if side32 is not None else None
            lp = sideplain.tick_end() if sideplain is not None else None
            due = (t in check_ticks) if check_ticks is not None else (t % check_every == 0)
            due = due or t == n_ticks - 1
            if not parallel or due:
                wo, vo, updates = main.state()
                if not np.isfinite(wo).all() or np.abs(wo).max() > finite_limit:
                    break
            tl = tol if loose_after is None or t < loose_after[0] else loose_after[1]
            if fragile_margin is not None:
                # a close call in the forward of (stage s, sample i) shows in the gradients
                # from that sample's backward at stage s on, at tick i + 2(S-1) - s
                o = main.o
                for s_ in range(S_):
                    if t - s_ >= 0 and o.min_margin.get((s_, t - s_), float("inf")) < fragile_margin:
                        effect = (t - s_) + 2 * (S_ - 1) - s_
                        fragile_tick = effect if fragile_tick is None else min(fragile_tick, effect)
                if fragile_tick is not None and t >= fragile_tick:
                    tl = max(tl, fragile_tol)
            if math.isnan(lo):
                assert math.isnan(lg), "tick %d: loss should be NaN while the pipeline fills" % t
            else:
                # loss = logsumexp(o) - o[label] is a difference of numbers of the
                # logits' size, so its rounding error scales with max|o|, not with itself
                mxl = main.last_max_logit
                e = abs(lg - lo) / max(abs(lo), mxl, 1e-12)
                worst["loss"] = max(worst["loss"], e)
                # flipped units move the trajectory, hence later losses (float32 runs: only once a
                # decision that either side may take differently is in play)
                ff = float(flip_floor.max()) if (fragile_margin is None or (fragile_tick is not None and t >= fragile_tick)) else 0.0
                tll = max(tl, ff)
                if lo32 is not None and not math.isnan(lo32):
                    # late in a long bfloat16 run two correct evaluations have drifted apart: the
                    # checker's own float32 run tells by how much (largest distance so far: the
                    # drift grows with the tick, a single tick's distance can be small by chance)
                    loss_spread = max(loss_spread, abs(lo32 - lo) / max(abs(lo), mxl, 1e-12))
                    tll = max(tll, 2 * spread_factor * loss_spread)      # (a single number per tick scatters more than a norm)
                assert e <= tll, "tick %d: loss %r vs %r (rel %.3g, bound %.3g)" % (t, lg, lo, e, tll)
                if abs(lo) > 1e-3 * mxl:
                    ep = abs(lg - lo) / abs(lo)
                    worst["plain_loss"] = max(worst["plain_loss"], ep)
                    if plain_loss_tol is not None:
                        tlp = max(plain_loss_tol, tl, ff)
                        if lo32 is not None and not math.isnan(lo32):
                            plain_spread = max(plain_spread, abs(lo32 - lo) / abs(lo))
                            tlp = max(tlp, 2 * spread_factor * plain_spread)
                        assert ep <= tlp, "tick %d: plain loss ratio %.3g (bound %.3g)" % (t, ep, tlp)
                if lp is not None and not math.isnan(lp):
                    eu = abs(lg - lp) / max(abs(lp), 1e-12)
                    worst["unrounded_loss"] = max(worst["unrounded_loss"], eu)
                    assert eu <= unrounded_loss_tol, \
                        "tick %d: loss %r vs %r of the checker without operand rounding (rel %.3g)" % (t, lg, lp, eu)
            if due:
                tw = tv = tl
                if side32 is not None:
                    w32, v32, _ = side32.state()
                    sp = tensor_spread(slices, w32, v32, wo, vo, w_init)
                    # a stage's gradient is made from everything downstream of it
                    stage_sp = np.zeros((S_, 2))
                    for (s_, _k), (a, b) in sp.items():
                        stage_sp[s_, 0] = max(stage_sp[s_, 0], a)
                        stage_sp[s_, 1] = max(stage_sp[s_, 1], b)
                    down = np.maximum.accumulate(stage_sp[::-1], axis=0)[::-1]
                    tw = {(s_, k_): max(tl, spread_factor * down[s_, 0], flip_floor[s_]) for s_, k_, _ in slices}
                    tv = {(s_, k_): max(tl, spread_factor * down[s_, 1], flip_floor[s_]) for s_, k_, _ in slices}
                elif flip_allowance is not None and (fragile_margin is None or (fragile_tick is not None and t >= fragile_tick)):
                    # (float32 runs: only once a decision that either side may take differently is in play)
                    tw = tv = {(s_, k_): max(tl, flip_floor[s_]) for s_, k_, _ in slices}
                ge_w, ge_v = eng.get_weights(), eng.get_velocity()
                if check_update_rule:
                    if prev_state is not None and prev_state[0] == t - 1:
                        r = update_rule_residual(meta, slices, prev_state[1], prev_state[2], ge_w, ge_v)
                        worst["update_rule"] = max(worst["update_rule"], r)
                        assert r <= 1.0, "tick %d: the engine's own step does not follow w <- w - lr (a v + b g) (ratio %.3g)" % (t, r)
                    prev_state = (t, ge_w, ge_v)
                rw, rv, fails = compare_state(slices, w_init, ge_w, ge_v, wo, vo, updates, tw, tv)
                assert not fails, "tick %d: %s" % (t, "; ".join(fails[:6]))
                worst["w"], worst["v"] = max(worst["w"], rw * tl), max(worst["v"], rv * tl)
                if fragile_tick is None or t < fragile_tick:
                    worst["strict_w"], worst["strict_v"] = max(worst["strict_w"], rw * tl), max(worst["strict_v"], rv * tl)
                worst["min_updates"] = min(updates)
            worst["ticks"] = t + 1
            worst["fragile_tick"] = fragile_tick
    finally:
        for q in sides:
            q.close()
    eng.destroy()
    return worst
