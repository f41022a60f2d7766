"""Shared helpers of the GPU parity tests: run the CUDA engine and the CPU
checker on the same seeded inputs and compare per tick."""
import math

import numpy as np

from oracle import PBOracle
from pb_workloads import he_normal_weights, make_inputs


def rel_err(got, ref):
    """||got - ref||_2 / max(||ref||_2, 1e-12); tensors that are exactly zero
    in the reference must be exactly zero."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    n = np.linalg.norm(ref)
    if n == 0.0:
        return 0.0 if not got.any() else float("inf")
    return float(np.linalg.norm(got - ref) / max(n, 1e-12))


def make_oracle(wl, dtype=np.float64, **kw):
    if wl.flags & 8:
        kw.setdefault("conv_operands", "bf16")
    o = PBOracle(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum,
                 wl.flags & 7, dtype=dtype, **kw)
    o.set_weights(he_normal_weights(wl.seed, wl))
    return o


def make_engine(wl):
    import torch
    from paper_2003_11666_b200 import PB
    eng = PB(wl.layers, wl.stage_of_layer, wl.in_shape, wl.n_classes, wl.lr, wl.momentum,
             wl.flags, stream=torch.cuda.current_stream().cuda_stream)
    eng.set_weights(he_normal_weights(wl.seed, wl))
    return eng


def compare_ticks(wl, n_ticks, tol, check_every=1, finite_limit=1e30, loose_after=None,
                  fragile_margin=None, fragile_tol=None, spread_factor=None, mitigation=None):
    """Tick both sides one sample at a time; returns the worst errors seen.

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
    bound on weights and velocities at a tick becomes
    max(tol, spread_factor * distance between its float32 and float64 runs)."""
    import torch
    x, y = make_inputs(wl.seed, n_ticks, wl.sample_elems, wl.n_classes)
    okw = {}
    if mitigation is not None:       # (SC delay scale, LWP horizon scale), e.g. (2, 2) for SC_2D + LWP_2D
        okw = dict(sc_delay_scale=mitigation[0], horizon_scale=mitigation[1])
    o = make_oracle(wl, margins=fragile_margin is not None, **okw)
    fragile_tick = None
    o32 = make_oracle(wl, dtype=np.float32, **okw) if spread_factor is not None else None
    eng = make_engine(wl)
    if mitigation is not None:
        eng.set_mitigation(*mitigation)
    xd = torch.from_numpy(x).cuda()
    worst = {"loss": 0.0, "w": 0.0, "v": 0.0, "ticks": 0, "fragile_tick": None, "strict_w": 0.0, "strict_v": 0.0}
    for t in range(n_ticks):
        lo = o.tick(x[t], y[t])
        lg = eng.tick(xd[t], int(y[t]))
        if o32 is not None:
            o32.tick(x[t], y[t])
        wo = o.get_weights()
        if not np.isfinite(wo).all() or np.abs(wo).max() > finite_limit:
            break
        tl = tol if loose_after is None or t < loose_after[0] else loose_after[1]
        if fragile_margin is not None:
            # a close call in the forward of (stage s, sample i) shows in the gradients
            # from that sample's backward at stage s on, at tick i + 2(S-1) - s
            for s_ in range(o.S):
                if t - s_ >= 0 and o.min_margin.get((s_, t - s_), float("inf")) < fragile_margin:
                    effect = (t - s_) + 2 * (o.S - 1) - s_
                    fragile_tick = effect if fragile_tick is None else min(fragile_tick, effect)
            if fragile_tick is not None and t >= fragile_tick:
                tl = max(tl, fragile_tol)
        if math.isnan(lo):
            assert math.isnan(lg), "tick %d: loss should be NaN while the pipeline fills" % t
        else:
            # loss = logsumexp(o) - o[label] is a difference of numbers of the
            # logits' size, so its rounding error scales with max|o|, not with itself
            e = abs(lg - lo) / max(abs(lo), float(np.abs(o.last_logits).max()), 1e-12)
            worst["loss"] = max(worst["loss"], e)
            assert e <= tl, "tick %d: loss %r vs %r (rel %.3g)" % (t, lg, lo, e)
        if t % check_every == 0 or t == n_ticks - 1:
            ew = rel_err(eng.get_weights(), wo)
            ev = rel_err(eng.get_velocity(), o.get_velocity())
            tlw = tlv = tl
            if o32 is not None:
                tlw = max(tl, spread_factor * rel_err(o32.get_weights(), wo))
                tlv = max(tl, spread_factor * rel_err(o32.get_velocity(), o.get_velocity()))
            worst["w"], worst["v"] = max(worst["w"], ew), max(worst["v"], ev)
            if fragile_tick is None or t < fragile_tick:
                worst["strict_w"], worst["strict_v"] = max(worst["strict_w"], ew), max(worst["strict_v"], ev)
            assert ew <= tlw, "tick %d: weights rel err %.3g (bound %.3g)" % (t, ew, tlw)
            assert ev <= tlv, "tick %d: velocity rel err %.3g (bound %.3g)" % (t, ev, tlv)
        worst["ticks"] = t + 1
        worst["fragile_tick"] = fragile_tick
    eng.destroy()
    return worst
